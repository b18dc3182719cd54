// Building blocks shared by the tensor-core kernels (importance passes, prefill attention):
// bounded mbarrier waits, TMA tile loads, tcgen05 MMA / TMEM access in inline PTX, the causal
// geometry with a visible prefix and the host-side tensor-map encoding.
#pragma once

#include "ec_common.cuh"

#include <cuda.h>

namespace ec {

namespace {

constexpr int kTileRows = 128;            // rows of a tile = MMA M
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // 1 s per wait, then give up
constexpr unsigned kPollBackoffNs = 32;                      // sleep between polls of the TMA / MMA threads


__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// Bounded wait. Returns false when the CTA is aborting or the time limit passed (in which
// case the abort flag and the global status word are set).
// `backoff_ns` > 0 makes the poller sleep between attempts: used by the single-thread TMA and MMA
// roles so that their polling does not take issue slots from the softmax warps of the same SM.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status,
                                          unsigned long long limit_ns = kWaitLimitNs, unsigned backoff_ns = 0)
{
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t spin = 1;; ++spin) {
        if (backoff_ns) __nanosleep(backoff_ns);
        if (mbar_try(bar, parity)) return true;
        if ((spin & 63u) == 0) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > limit_ns) {
                *abort_flag = 1;
                atomicExch(status, 1);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
                 " [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}

// K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// D = A * B^T, A and B bf16 K-major in shared memory, fp32 accumulator in TMEM, M = N = 128, K = 16.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive fp32 columns of this thread's TMEM lane; the data is valid after tmem_ld_wait.
__device__ __forceinline__ void tmem_ld32_async(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
}

// Waits for every outstanding TMEM load of this thread; the registers of `r` are marked as
// redefined here so that no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) asm volatile("" : "+r"(r[i]));
}

// One ex2 per score element makes the special-function unit the busiest pipe of these kernels
// (16 results per clock per SM). One element pair in EC_IMP_POLY_PAIR_EVERY is therefore evaluated
// on the FMA pipe instead, with packed fp32 pair instructions: Cody-Waite split and a degree-4
// polynomial, relative error < 6e-6, inputs clamped at -125 (so a masked -inf gives 2^-125, far
// below one ulp of any sum it joins). Measured on B200: +3% at T = 640, +6-8% at T >= 2048 with
// one pair in four; one in three or two is slower again. 0 turns it off.
#ifndef EC_IMP_POLY_PAIR_EVERY
#define EC_IMP_POLY_PAIR_EVERY 4
#endif
__device__ __forceinline__ float2 poly_exp2_pair(float2 x)
{
    const float2 magic = make_float2(12582912.f, 12582912.f);       // 1.5 * 2^23: low mantissa bits = round(x)
    const float2 nmagic = make_float2(-12582912.f, -12582912.f), neg1 = make_float2(-1.f, -1.f);
    x.x = fmaxf(x.x, -125.f);
    x.y = fmaxf(x.y, -125.f);
    const float2 t = __fadd2_rn(x, magic);
    const float2 f = __ffma2_rn(__fadd2_rn(t, nmagic), neg1, x);    // fractional part in [-0.5, 0.5]
    float2 p = __ffma2_rn(f, make_float2(0.00935919489711523f, 0.00935919489711523f),
                          make_float2(0.05588679388165474f, 0.05588679388165474f));
    p = __ffma2_rn(p, f, make_float2(0.2402936965227127f, 0.2402936965227127f));
    p = __ffma2_rn(p, f, make_float2(0.6931265592575073f, 0.6931265592575073f));
    p = __ffma2_rn(p, f, make_float2(0.9999980926513672f, 0.9999980926513672f));
    return make_float2(__int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23)),   // scale by 2^round(x)
                       __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23)));
}

// 2^a for a pair; `pair_index` is a compile-time constant after unrolling.
__device__ __forceinline__ float2 exp2_pair(float2 a, int pair_index)
{
    constexpr int every = EC_IMP_POLY_PAIR_EVERY > 0 ? EC_IMP_POLY_PAIR_EVERY : 1;
    if (EC_IMP_POLY_PAIR_EVERY > 0 && pair_index % every == 0) return poly_exp2_pair(a);
    return make_float2(fast_exp2(a.x), fast_exp2(a.y));
}

// part[k] += 2^(v*c - m) over the 32 values of a chunk, two elements per instruction: the
// scale-and-shift and the accumulation are packed fp32 pairs, only the ex2 itself is scalar.
// Element i lands in chain i & 3, as a scalar loop over four chains would put it.
__device__ __forceinline__ void sum_exp2(const float (&v)[32], float c, float m, float2 (&part)[2])
{
    const float2 c2 = make_float2(c, c), nm = make_float2(-m, -m);
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        const float2 a = __ffma2_rn(make_float2(v[i], v[i + 1]), c2, nm);
        part[(i >> 1) & 1] = __fadd2_rn(part[(i >> 1) & 1], exp2_pair(a, i >> 1));
    }
}

// Geometry of the causal contraction with a visible prefix: query m sees keys n <= m + P.
struct Geometry {
    int Tq, P, ntq, ntk;
    __host__ __device__ int Tk() const { return Tq + P; }
    // pass 1: last key tile a query tile touches
    __host__ __device__ int jmax(int i) const { int j = (i * kTileRows + kTileRows - 1 + P) / kTileRows; return j < ntk - 1 ? j : ntk - 1; }
    // pass 2: first query tile that sees a key tile
    __host__ __device__ int imin(int j) const { int d = j * kTileRows - P; return d > 0 ? d / kTileRows : 0; }
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// [units, T, D] bf16 seen as a 3-D tensor; a box is 64 columns (128 bytes) x 128 rows of one unit.
// Rows past T read as zeros, so ragged prompts need no host-side padding.
inline bool make_map(CUtensorMap *map, const void *ptr, int units, int T, int D)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)T, (cuuint64_t)units};
    cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)T * D * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)kTileRows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline int sm_count()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 148;
    return n;
}


}  // namespace

}  // namespace ec
