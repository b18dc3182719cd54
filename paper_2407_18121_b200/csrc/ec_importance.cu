// Importance of every prompt key (Sec. 3.3, Eq. 1 and the column sums that follow it),
// computed in two passes so that the T x T attention matrix is never stored:
//   pass 1: lse[m]   = log2 sum_{n<=m} 2^(c*<q_m,k_n>)          c = scale*log2(e)
//   pass 2: score[n] = sum_{m>=n} 2^(c*<q_m,k_n> - lse[m])
// Both passes are the same dense causal contraction, run on the 5th-generation tensor
// cores: 128x128 score tiles are produced by tcgen05.mma from TMA-staged bf16 tiles into
// TMEM, and read back one row per thread, so a thread owns a query row in pass 1 and a key
// row in pass 2 and every reduction stays inside a thread (no atomics, run-to-run identical).
//
// One CTA owns a "stationary" 128-row tile of one unit and streams the other operand's tiles
// past it. Warp roles: warp 0 issues TMA loads, warp 1 issues MMAs and owns the TMEM
// allocation, warps 2..5 (one thread per TMEM lane) do the softmax arithmetic.
// Every mbarrier wait is bounded in time; on expiry the CTA records a status word and leaves.
#include "ec_common.cuh"

#include <cuda.h>

namespace ec {

namespace {

constexpr int kTileRows = 128;            // rows of a tile = MMA M = MMA N
constexpr int kThreads = 192;             // 6 warps: TMA, MMA, 4 x softmax
constexpr int kAccBufs = 2;               // TMEM accumulator buffers (128 columns each)
constexpr int kTmemCols = 256;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // 1 s per wait, then give up

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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status,
                                          unsigned long long limit_ns = kWaitLimitNs)
{
    if (mbar_try(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (uint32_t spin = 1;; ++spin) {
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

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32])
{
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

template <int D, int STAGES>
struct Smem {
    static constexpr int kTileBytes = kTileRows * D * 2;
    static constexpr int kStat = 0;
    static constexpr int kStage0 = kTileBytes;
    static constexpr int kLse = kStage0 + STAGES * kTileBytes;            // 2 x 128 floats
    static constexpr int kBars = kLse + kAccBufs * kTileRows * 4;
    // barrier slots (8 bytes each): stat_full, full[STAGES], empty[STAGES], acc_full[2], acc_empty[2], lse_ready[2]
    static constexpr int kNumBars = 1 + 2 * STAGES + 3 * kAccBufs;
    static constexpr int kTmemSlot = kBars + kNumBars * 8;
    static constexpr int kAbort = kTmemSlot + 4;
    static constexpr int kTotal = kAbort + 4;
    static constexpr int kDynBytes = kTotal + 1024;                       // slack for 1024-byte alignment
};

// PASS2 == false: stationary = query tile i, streamed = key tiles i, i-1, .., 0   -> lse2 (and lse_out)
// PASS2 == true : stationary = key tile j,   streamed = query tiles j, j+1, .., nt-1 -> scores
// The first streamed tile is always the diagonal one (the only tile that needs the causal mask).
// lse2 is padded to nt*128 entries per unit; entries past T hold +inf so that pass 2 gives
// those (non-existent) queries zero weight.
template <int D, int STAGES, bool PASS2>
__global__ void __launch_bounds__(kThreads, 2)
importance_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  int T, int nt, float c, float *__restrict__ lse2, float *__restrict__ lse_out,
                  float *__restrict__ scores, int *__restrict__ status)
{
    using L = Smem<D, STAGES>;
    constexpr int kTileBytes = L::kTileBytes;
    constexpr int kBoxes = D / 64;                          // TMA boxes (64 bf16 = 128 B wide) per tile
    constexpr int kBoxBytes = kTileRows * 128;
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((kTileRows >> 3) << 17) | ((kTileRows >> 4) << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + L::kBars;
    const uint32_t bar_stat = bars;
    auto bar_full = [&](int s) { return bars + 8u * (1 + s); };
    auto bar_empty = [&](int s) { return bars + 8u * (1 + STAGES + s); };
    auto bar_acc_full = [&](int b) { return bars + 8u * (1 + 2 * STAGES + b); };
    auto bar_acc_empty = [&](int b) { return bars + 8u * (1 + 2 * STAGES + kAccBufs + b); };
    auto bar_lse = [&](int b) { return bars + 8u * (1 + 2 * STAGES + 2 * kAccBufs + b); };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(base_ptr + L::kTmemSlot);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(base_ptr + L::kAbort);
    float *lse_s = reinterpret_cast<float *>(base_ptr + L::kLse);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int unit = blockIdx.x / nt;
    const int w = blockIdx.x - unit * nt;                   // heaviest tile of the unit first
    const int stat_tile = PASS2 ? w : nt - 1 - w;
    const int count = PASS2 ? nt - stat_tile : stat_tile + 1;
    const CUtensorMap *map_stat = PASS2 ? &map_k : &map_q;
    const CUtensorMap *map_strm = PASS2 ? &map_q : &map_k;

    // a CTA of this launch has already given up: leave at once instead of timing out again
    if (threadIdx.x == 0) *abort_flag = *reinterpret_cast<volatile int *>(status);
    __syncthreads();
    if (*abort_flag) return;

    if (threadIdx.x == 0) {
        mbar_init(bar_stat, 1);
        for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(bar_acc_full(b), 1);
            mbar_init(bar_acc_empty(b), 4);
            mbar_init(bar_lse(b), 4 * 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + (uint32_t)L::kTmemSlot), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            mbar_expect_tx(bar_stat, kTileBytes);
#pragma unroll
            for (int bx = 0; bx < kBoxes; ++bx)
                tma_load_3d(base + L::kStat + bx * kBoxBytes, map_stat, bx * 64, stat_tile * kTileRows, unit, bar_stat);
            int armed = 0;
            for (int t = 0; t < count; ++t) {
                const int s = t % STAGES;
                const uint32_t ph = (uint32_t)(t / STAGES) & 1u;
                if (!mbar_wait(bar_empty(s), ph ^ 1u, abort_flag, status)) break;
                const int tile = PASS2 ? stat_tile + t : stat_tile - t;
                mbar_expect_tx(bar_full(s), kTileBytes);
#pragma unroll
                for (int bx = 0; bx < kBoxes; ++bx)
                    tma_load_3d(base + L::kStage0 + s * kTileBytes + bx * kBoxBytes, map_strm, bx * 64,
                                tile * kTileRows, unit, bar_full(s));
                armed = t + 1;
            }
            if (*abort_flag) {
                // let copies that are still in flight land before the CTA gives its memory back
                mbar_wait(bar_stat, 0, abort_flag, status, 200000ull);
                for (int t = max(0, armed - STAGES); t < armed; ++t)
                    mbar_wait(bar_full(t % STAGES), (uint32_t)(t / STAGES) & 1u, abort_flag, status, 200000ull);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            bool ok = mbar_wait(bar_stat, 0, abort_flag, status);
            for (int t = 0; ok && t < count; ++t) {
                const int s = t % STAGES, b = t % kAccBufs;
                const uint32_t ph = (uint32_t)(t / STAGES) & 1u, bph = (uint32_t)(t / kAccBufs) & 1u;
                if (!mbar_wait(bar_acc_empty(b), bph ^ 1u, abort_flag, status)) break;
                if (!mbar_wait(bar_full(s), ph, abort_flag, status)) break;
                tc_fence_after();
                const uint32_t a0 = base + L::kStat, b0 = base + L::kStage0 + s * kTileBytes;
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (uint32_t)(k / 4) * kBoxBytes + (uint32_t)(k % 4) * 32u;
                    umma_bf16(tmem_base + (uint32_t)b * kTileRows, umma_desc(a0 + off), umma_desc(b0 + off), kIdesc,
                              k > 0 ? 1u : 0u);
                }
                umma_commit(bar_empty(s));       // stage reusable once these MMAs have read it
                umma_commit(bar_acc_full(b));    // accumulator ready for the softmax warps
            }
        }
    } else {
        // ---------------------------------------------------------------- softmax warps
        const int q4 = warp & 3;                              // TMEM lane quarter this warp may read
        const int r = q4 * 32 + lane;                         // row of the stationary tile = TMEM lane
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16);
        const size_t lse_row = (size_t)unit * nt * kTileRows;
        float mrun = -INFINITY, Z = 0.f;                      // pass 1 running max / sum (log2 domain)
        float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f; // pass 2 column sum
        bool ok = true;
        for (int t = 0; t < count; ++t) {
            const int b = t % kAccBufs;
            const uint32_t bph = (uint32_t)(t / kAccBufs) & 1u;
            if (PASS2) {
                const int tile = stat_tile + t;
                // every softmax thread stages one entry of the tile's lse, then all wait (bounded) for
                // the 128 entries; the buffer is reused two tiles later, after the next tile's rendezvous
                lse_s[b * kTileRows + r] = lse2[lse_row + (size_t)tile * kTileRows + r];
                mbar_arrive(bar_lse(b));
                if (!mbar_wait(bar_lse(b), bph, abort_flag, status)) { ok = false; break; }
            }
            if (!mbar_wait(bar_acc_full(b), bph, abort_flag, status)) { ok = false; break; }
            tc_fence_after();
            const bool diag = (t == 0);
#pragma unroll 1
            for (int ch = 0; ch < kTileRows / 32; ++ch) {
                float v[32];
                tmem_ld32(lane_addr + (uint32_t)(b * kTileRows + ch * 32), v);
                if (!PASS2) {
                    if (diag) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) if (ch * 32 + i > r) v[i] = -INFINITY;   // key n <= query m
                    }
                    float cm = v[0];
#pragma unroll
                    for (int i = 1; i < 32; ++i) cm = fmaxf(cm, v[i]);
                    const float mnew = fmaxf(mrun, cm * c);
                    if (mnew != -INFINITY) {
                        float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int i = 0; i < 32; ++i) part[i & 3] += fast_exp2(fmaf(v[i], c, -mnew));
                        Z = Z * fast_exp2(mrun - mnew) + ((part[0] + part[1]) + (part[2] + part[3]));
                        mrun = mnew;
                    }
                } else {
                    const float4 *ls = reinterpret_cast<const float4 *>(lse_s + b * kTileRows + ch * 32);
#pragma unroll
                    for (int i4 = 0; i4 < 8; ++i4) {
                        const float4 l4 = ls[i4];
                        float p0 = fast_exp2(fmaf(v[i4 * 4 + 0], c, -l4.x));
                        float p1 = fast_exp2(fmaf(v[i4 * 4 + 1], c, -l4.y));
                        float p2 = fast_exp2(fmaf(v[i4 * 4 + 2], c, -l4.z));
                        float p3 = fast_exp2(fmaf(v[i4 * 4 + 3], c, -l4.w));
                        if (diag) {                                                       // query m >= key n
                            const int c0 = ch * 32 + i4 * 4;
                            if (c0 + 0 < r) p0 = 0.f;
                            if (c0 + 1 < r) p1 = 0.f;
                            if (c0 + 2 < r) p2 = 0.f;
                            if (c0 + 3 < r) p3 = 0.f;
                        }
                        acc0 += p0; acc1 += p1; acc2 += p2; acc3 += p3;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty(b));
        }
        if (ok) {
            const int row = stat_tile * kTileRows + r;
            if (!PASS2) {
                const float l2 = (row < T) ? mrun + __log2f(Z) : INFINITY;
                lse2[lse_row + row] = l2;
                if (lse_out && row < T) lse_out[(size_t)unit * T + row] = l2 * kLn2;
            } else if (row < T) {
                scores[(size_t)unit * T + row] = (acc0 + acc1) + (acc2 + acc3);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
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
bool make_map(CUtensorMap *map, const void *ptr, int units, int T, int D)
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

// A caller-provided natural-log normaliser [units, T] -> the padded log2-domain layout pass 2 reads.
__global__ void lse_import_kernel(const float *__restrict__ lse_nat, float *__restrict__ lse2, int T, int Tpad)
{
    const int unit = blockIdx.y;
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= Tpad) return;
    lse2[(size_t)unit * Tpad + m] = (m < T) ? lse_nat[(size_t)unit * T + m] * kLog2e : INFINITY;
}

template <int D, int STAGES>
cudaError_t launch_passes(const CUtensorMap &mq, const CUtensorMap &mk, int units, int T, int nt, float c, float *lse2,
                          float *lse_out, float *scores, int *status, bool first_pass, cudaStream_t stream)
{
    constexpr int smem = Smem<D, STAGES>::kDynBytes;
    cudaError_t e = cudaFuncSetAttribute(importance_kernel<D, STAGES, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(importance_kernel<D, STAGES, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)units * (unsigned)nt;
    if (first_pass)
        importance_kernel<D, STAGES, false><<<grid, kThreads, smem, stream>>>(mq, mk, T, nt, c, lse2, lse_out, scores, status);
    importance_kernel<D, STAGES, true><<<grid, kThreads, smem, stream>>>(mq, mk, T, nt, c, lse2, lse_out, scores, status);
    return cudaGetLastError();
}

}  // namespace

size_t importance_workspace_bytes(int N, int H, int T, int D)
{
    (void)D;
    const size_t nt = (size_t)(T + kTileRows - 1) / kTileRows;
    return kStatusBytes + (size_t)N * H * nt * kTileRows * sizeof(float);   // status block + padded lse
}

// lse_in == nullptr: both passes. Otherwise the caller's normaliser replaces pass 1.
cudaError_t launch_importance(const void *Q, const void *K, float *scores, float *lse_out, const float *lse_in,
                              int N, int H, int T, int D, float scale, void *ws, cudaStream_t stream)
{
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return e;
    int *status = static_cast<int *>(ws);
    float *lse2 = reinterpret_cast<float *>(static_cast<char *>(ws) + kStatusBytes);
    const int units = N * H;
    const int nt = (T + kTileRows - 1) / kTileRows;
    if ((long long)units * nt > 0x7FFFFFFFLL || units > 65535 * 1024) return cudaErrorInvalidConfiguration;
    CUtensorMap mq, mk;
    if (!make_map(&mq, Q, units, T, D) || !make_map(&mk, K, units, T, D)) return cudaErrorInvalidValue;
    if (lse_in) {
        if (units > 65535) return cudaErrorInvalidConfiguration;
        dim3 g((nt * kTileRows + 255) / 256, units);
        lse_import_kernel<<<g, 256, 0, stream>>>(lse_in, lse2, T, nt * kTileRows);
    }
    const float c = scale * kLog2e;
    if (D == 128)
        return launch_passes<128, 2>(mq, mk, units, T, nt, c, lse2, lse_out, scores, status, lse_in == nullptr, stream);
    return launch_passes<64, 4>(mq, mk, units, T, nt, c, lse2, lse_out, scores, status, lse_in == nullptr, stream);
}

}  // namespace ec
