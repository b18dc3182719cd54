// Bucket division (Eq. 2) and mean merge (Eq. 3) into the dense compacted cache.
// HBM-bound streaming: every prompt row of K and V is read exactly once with 16-byte loads,
// every kept row is written once.
//
// Buckets are consecutive row ranges, so a run of buckets is one contiguous range of prompt
// rows. A CTA takes a slice of prompt rows of one unit; each lane group takes an equal part
// of the slice, owns the buckets that START inside its part, and streams their rows in order
// (addresses do not depend on the bucket structure, so many loads are in flight), flushing a
// mean whenever it passes a bucket's last row.
#include "ec_common.cuh"

namespace ec {

namespace {

#ifndef EC_MERGE_THREADS
#define EC_MERGE_THREADS 128
#endif
#ifndef EC_MERGE_ROWS_PER_CTA
#define EC_MERGE_ROWS_PER_CTA 256
#endif
#ifndef EC_MERGE_UNROLL
#define EC_MERGE_UNROLL 8
#endif
#ifndef EC_MERGE_MIN_CTAS
#define EC_MERGE_MIN_CTAS 8      // 64 registers: eight CTAs per SM (68 registers and seven CTAs without the bound)
#endif
constexpr int kMergeThreads = EC_MERGE_THREADS;
constexpr int kRowsPerCta = EC_MERGE_ROWS_PER_CTA;
constexpr int kUnroll = EC_MERGE_UNROLL;

__device__ __forceinline__ float2 unpack2(uint32_t w) { return make_float2(bf16lo(w), bf16hi(w)); }

// First row of bucket k (Eq. 2): one past the midpoint between anchors k-1 and k.
__device__ __forceinline__ int bucket_lo(const int32_t *anch, int k)
{
    return (k == 0) ? 0 : ((anch[k - 1] + anch[k]) >> 1) + 1;
}

// Smallest k in [0, C] whose bucket starts at or after row r (C when none does).
__device__ __forceinline__ int first_bucket_from(const int32_t *anch, int C, int r)
{
    int lo = 0, hi = C;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (bucket_lo(anch, mid) >= r) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// LPR = lanes per row = D / 8 (each lane holds 8 bf16 = 16 bytes of a row). A lane group is
// 2*LPR lanes: the first LPR stream the K row of a position, the other LPR its V row, so both
// halves see the same bucket boundaries (for D = 128 a group is exactly one warp: no divergence).
// grid.x = units * slices (equal slices of at most 256 rows). Dynamic shared memory: the unit's C anchors.
template <int LPR>
__global__ void __launch_bounds__(kMergeThreads, EC_MERGE_MIN_CTAS)
merge_kernel(const uint4 *__restrict__ K, const uint4 *__restrict__ V, const int32_t *__restrict__ anchor_pos,
             int T, int C, int slices, uint4 *__restrict__ Kc, uint4 *__restrict__ Vc, int cap)
{
    constexpr int GL = 2 * LPR;                     // lanes per group
    constexpr int G = kMergeThreads / GL;           // lane groups per CTA
    extern __shared__ int32_t anch[];
    const int unit = blockIdx.x / slices;
    const int slice = blockIdx.x - unit * slices;
    const int g = threadIdx.x / GL;
    const int gl = threadIdx.x - g * GL;
    const bool is_v = gl >= LPR;
    const int l = is_v ? gl - LPR : gl;

    // launched with programmatic stream serialization right behind the selection kernel:
    // wait for its anchors before the first global access
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int32_t *ap = anchor_pos + (size_t)unit * C;
    for (int k = threadIdx.x; k < C; k += kMergeThreads) anch[k] = ap[k];
    __syncthreads();

    const int slice_rows = (T + slices - 1) / slices;      // equal slices: at most kRowsPerCta rows each
    const int R0 = slice * slice_rows, R1 = min(R0 + slice_rows, T);
    const int part = (R1 - R0 + G - 1) / G;
    const int ra = min(R0 + g * part, R1), rb = min(ra + part, R1);
    int k = first_bucket_from(anch, C, ra);
    const int k_end = first_bucket_from(anch, C, rb);
    if (k >= k_end) return;

    const uint4 *src = (is_v ? V : K) + (size_t)unit * T * LPR + l;
    uint4 *dst = (is_v ? Vc : Kc) + (size_t)unit * cap * LPR + l;

    int lo = bucket_lo(anch, k);
    const int last = (k_end == C) ? T - 1 : bucket_lo(anch, k_end) - 1;   // last row this group reads
    int hi = (k == C - 1) ? T - 1 : ((anch[k] + anch[k + 1]) >> 1);
    const float2 one2 = make_float2(1.f, 1.f), zero2 = make_float2(0.f, 0.f);
    float2 acc[4];                                   // packed fp32 pairs: elements 2i, 2i+1 of this lane's 8
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i] = zero2;

    for (int t = lo; t <= last; t += kUnroll) {
        uint4 rw[kUnroll];
#pragma unroll
        for (int j = 0; j < kUnroll; ++j)            // rows past the range: reload the last row, unused
            rw[j] = ldg_stream(src + (size_t)min(t + j, last) * LPR);
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) {
            if (t + j <= last) {
                acc[0] = __ffma2_rn(unpack2(rw[j].x), one2, acc[0]);
                acc[1] = __ffma2_rn(unpack2(rw[j].y), one2, acc[1]);
                acc[2] = __ffma2_rn(unpack2(rw[j].z), one2, acc[2]);
                acc[3] = __ffma2_rn(unpack2(rw[j].w), one2, acc[3]);
                if (t + j == hi) {
                    const int cnt = hi - lo + 1;
                    const float inv = (cnt == 1) ? 1.0f : __frcp_rn((float)cnt);   // a singleton stays bit-exact
                    const float2 inv2 = make_float2(inv, inv);
                    uint4 o;
                    float2 m;
                    m = __ffma2_rn(acc[0], inv2, zero2); o.x = pack2(m.x, m.y);
                    m = __ffma2_rn(acc[1], inv2, zero2); o.y = pack2(m.x, m.y);
                    m = __ffma2_rn(acc[2], inv2, zero2); o.z = pack2(m.x, m.y);
                    m = __ffma2_rn(acc[3], inv2, zero2); o.w = pack2(m.x, m.y);
                    dst[(size_t)k * LPR] = o;
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[i] = zero2;
                    ++k;
                    lo = hi + 1;
                    hi = (k >= C - 1) ? T - 1 : ((anch[k] + anch[k + 1]) >> 1);
                }
            }
        }
    }
}

// Eviction instead of merging: cache row k is the anchor's own row (everything else is dropped).
// One lane group per kept row; grid.x = units * ceil(C / groups per CTA).
template <int LPR>
__global__ void __launch_bounds__(kMergeThreads)
gather_kernel(const uint4 *__restrict__ K, const uint4 *__restrict__ V, const int32_t *__restrict__ anchor_pos,
              int T, int C, int chunks, uint4 *__restrict__ Kc, uint4 *__restrict__ Vc, int cap)
{
    constexpr int GL = 2 * LPR;
    constexpr int G = kMergeThreads / GL;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int unit = blockIdx.x / chunks;
    const int chunk = blockIdx.x - unit * chunks;
    const int g = threadIdx.x / GL, gl = threadIdx.x - g * GL;
    const bool is_v = gl >= LPR;
    const int l = is_v ? gl - LPR : gl;
    const int k = chunk * G + g;
    if (k >= C) return;
    const int t = anchor_pos[(size_t)unit * C + k];
    const uint4 *src = (is_v ? V : K) + ((size_t)unit * T + t) * LPR + l;
    uint4 *dst = (is_v ? Vc : Kc) + ((size_t)unit * cap + k) * LPR + l;
    *dst = ldg_stream(src);
}

// History for a further instruction: output row j of a unit is cache row j in queue order for
// j < P, new row j - P after it. One lane group per output row, K on its first half, V on the second.
// The launch covers output rows row0 .. P + Tq - 1.
template <int LPR>
__global__ void __launch_bounds__(kMergeThreads)
concat_kernel(const uint4 *__restrict__ Kc, const uint4 *__restrict__ Vc, int cap, int P, int base, int ring,
              int ring_head, const uint4 *__restrict__ K_new, const uint4 *__restrict__ V_new, int Tq, int row0, int chunks,
              uint4 *__restrict__ K_all, uint4 *__restrict__ V_all)
{
    constexpr int GL = 2 * LPR;
    constexpr int G = kMergeThreads / GL;
    const int unit = blockIdx.x / chunks;
    const int chunk = blockIdx.x - unit * chunks;
    const int g = threadIdx.x / GL, gl = threadIdx.x - g * GL;
    const bool is_v = gl >= LPR;
    const int l = is_v ? gl - LPR : gl;
    const int j = row0 + chunk * G + g;
    const int T = P + Tq;
    if (j >= T) return;
    const uint4 *src;
    if (j < P) {
        const int slot = (j < base || ring == 0) ? j : base + (ring_head + (j - base)) % ring;
        src = (is_v ? Vc : Kc) + ((size_t)unit * cap + slot) * LPR + l;
    } else {
        src = (is_v ? V_new : K_new) + ((size_t)unit * Tq + (j - P)) * LPR + l;
    }
    uint4 *dst = (is_v ? V_all : K_all) + ((size_t)unit * T + j) * LPR + l;
    *dst = ldg_stream(src);
}

// Cache rows whose slots follow no formula (retention-ratio policy): output rows j0 .. j0 + n - 1 of
// every unit come from the slots listed in `tab`, which travels by value in the kernel's parameters.
constexpr int kSlotTableRows = 896;
struct SlotTable { int slot[kSlotTableRows]; };

template <int LPR>
__global__ void __launch_bounds__(kMergeThreads)
concat_listed_kernel(const uint4 *__restrict__ Kc, const uint4 *__restrict__ Vc, int cap, int T_out, int j0, int n,
                     const __grid_constant__ SlotTable tab, int chunks, uint4 *__restrict__ K_all, uint4 *__restrict__ V_all)
{
    constexpr int GL = 2 * LPR;
    constexpr int G = kMergeThreads / GL;
    const int unit = blockIdx.x / chunks;
    const int chunk = blockIdx.x - unit * chunks;
    const int g = threadIdx.x / GL, gl = threadIdx.x - g * GL;
    const bool is_v = gl >= LPR;
    const int l = is_v ? gl - LPR : gl;
    const int j = chunk * G + g;
    if (j >= n) return;
    const uint4 *src = (is_v ? Vc : Kc) + ((size_t)unit * cap + tab.slot[j]) * LPR + l;
    uint4 *dst = (is_v ? V_all : K_all) + ((size_t)unit * T_out + j0 + j) * LPR + l;
    *dst = ldg_stream(src);
}

template <int LPR>
cudaError_t launch_merge_t(const void *K, const void *V, const int32_t *anchor_pos, unsigned grid, int T, int n_keep,
                           int slices, void *Kc, void *Vc, int cap, cudaStream_t stream)
{
    const size_t smem = (size_t)n_keep * sizeof(int32_t);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(merge_kernel<LPR>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kMergeThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, merge_kernel<LPR>, (const uint4 *)K, (const uint4 *)V, anchor_pos, T, n_keep, slices,
                              (uint4 *)Kc, (uint4 *)Vc, cap);
}

template <int LPR>
cudaError_t launch_gather_t(const void *K, const void *V, const int32_t *anchor_pos, int units, int T, int n_keep,
                            void *Kc, void *Vc, int cap, cudaStream_t stream)
{
    constexpr int G = kMergeThreads / (2 * LPR);
    const int chunks = (n_keep + G - 1) / G;
    if ((long long)units * chunks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(units * chunks));
    cfg.blockDim = dim3(kMergeThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gather_kernel<LPR>, (const uint4 *)K, (const uint4 *)V, anchor_pos, T, n_keep, chunks,
                              (uint4 *)Kc, (uint4 *)Vc, cap);
}

template <int LPR>
cudaError_t launch_concat_t(const void *Kc, const void *Vc, int units, int cap, int P, int base, int ring, int ring_head,
                            const void *K_new, const void *V_new, int Tq, int row0, void *K_all, void *V_all,
                            cudaStream_t stream)
{
    constexpr int G = kMergeThreads / (2 * LPR);
    const int chunks = (P + Tq - row0 + G - 1) / G;
    if ((long long)units * chunks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    concat_kernel<LPR><<<(unsigned)(units * chunks), kMergeThreads, 0, stream>>>(
        (const uint4 *)Kc, (const uint4 *)Vc, cap, P, base, ring, ring_head, (const uint4 *)K_new, (const uint4 *)V_new, Tq,
        row0, chunks, (uint4 *)K_all, (uint4 *)V_all);
    return cudaGetLastError();
}

template <int LPR>
cudaError_t launch_concat_listed_t(const void *Kc, const void *Vc, int units, int cap, int P, const int *slots,
                                   const void *K_new, const void *V_new, int Tq, void *K_all, void *V_all,
                                   cudaStream_t stream)
{
    constexpr int G = kMergeThreads / (2 * LPR);
    // the new rows: the plain kernel from output row P on
    cudaError_t e = launch_concat_t<LPR>(Kc, Vc, units, cap, P, P, 0, 0, K_new, V_new, Tq, P, K_all, V_all, stream);
    if (e != cudaSuccess) return e;
    for (int j0 = 0; j0 < P; j0 += kSlotTableRows) {
        const int n = P - j0 < kSlotTableRows ? P - j0 : kSlotTableRows;
        SlotTable tab;
        for (int j = 0; j < n; ++j) tab.slot[j] = slots[j0 + j];
        for (int j = n; j < kSlotTableRows; ++j) tab.slot[j] = 0;
        const int chunks = (n + G - 1) / G;
        if ((long long)units * chunks > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
        concat_listed_kernel<LPR><<<(unsigned)(units * chunks), kMergeThreads, 0, stream>>>(
            (const uint4 *)Kc, (const uint4 *)Vc, cap, P + Tq, j0, n, tab, chunks, (uint4 *)K_all, (uint4 *)V_all);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace

cudaError_t launch_merge(const void *K, const void *V, const int32_t *anchor_pos, int units, int T, int D,
                         int n_keep, void *Kc, void *Vc, int cap, cudaStream_t stream)
{
    const int slices = (T + kRowsPerCta - 1) / kRowsPerCta;
    const long long grid = (long long)units * slices;
    if (grid > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    if (D == 128) return launch_merge_t<16>(K, V, anchor_pos, (unsigned)grid, T, n_keep, slices, Kc, Vc, cap, stream);
    return launch_merge_t<8>(K, V, anchor_pos, (unsigned)grid, T, n_keep, slices, Kc, Vc, cap, stream);
}

cudaError_t launch_gather(const void *K, const void *V, const int32_t *anchor_pos, int units, int T, int D,
                          int n_keep, void *Kc, void *Vc, int cap, cudaStream_t stream)
{
    if (D == 128) return launch_gather_t<16>(K, V, anchor_pos, units, T, n_keep, Kc, Vc, cap, stream);
    return launch_gather_t<8>(K, V, anchor_pos, units, T, n_keep, Kc, Vc, cap, stream);
}

cudaError_t launch_concat(const void *Kc, const void *Vc, int units, int cap, int D, int P, int base, int ring,
                          int ring_head, const void *K_new, const void *V_new, int Tq, void *K_all, void *V_all,
                          cudaStream_t stream)
{
    if (D == 128)
        return launch_concat_t<16>(Kc, Vc, units, cap, P, base, ring, ring_head, K_new, V_new, Tq, 0, K_all, V_all, stream);
    return launch_concat_t<8>(Kc, Vc, units, cap, P, base, ring, ring_head, K_new, V_new, Tq, 0, K_all, V_all, stream);
}

cudaError_t launch_concat_listed(const void *Kc, const void *Vc, int units, int cap, int D, int P, const int *slots_host,
                                 const void *K_new, const void *V_new, int Tq, void *K_all, void *V_all,
                                 cudaStream_t stream)
{
    if (D == 128)
        return launch_concat_listed_t<16>(Kc, Vc, units, cap, P, slots_host, K_new, V_new, Tq, K_all, V_all, stream);
    return launch_concat_listed_t<8>(Kc, Vc, units, cap, P, slots_host, K_new, V_new, Tq, K_all, V_all, stream);
}

}  // namespace ec
