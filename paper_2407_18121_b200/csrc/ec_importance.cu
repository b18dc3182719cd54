// Importance of every prompt key (Sec. 3.3, Eq. 1 and the column sums that follow it),
// computed in two passes so that the attention matrix is never stored:
//   pass 1: lse[m]   = log2 sum_{n<=m+P} 2^(c*<q_m,k_n>)          c = scale*log2(e)
//   pass 2: score[n] = sum_{m>=n-P} 2^(c*<q_m,k_n> - lse[m])
// P is the number of keys that precede the first query (0 for a plain prompt; the rows of
// an earlier, already compacted cache when a new instruction is encoded on top of it).
// Both passes are the same dense causal contraction, run on the 5th-generation tensor
// cores: 128x128 score tiles are produced by tcgen05.mma from TMA-staged bf16 tiles into
// TMEM, and read back one row per thread, so a thread owns a query row in pass 1 and a key
// row in pass 2 and every reduction stays inside a thread (no atomics, run-to-run identical).
//
// A work item is a "stationary" 128-row tile of one unit, past which the other operand's
// tiles are streamed. CTAs are persistent (two per SM) and keep their barriers, TMEM
// allocation and TMA ring alive across items. Items are handed out in order (units in order
// for L2 reuse, a unit's tiles from the longest to the shortest) from a counter in global
// memory: a CTA's first item is its block index, every later one comes from an atomic
// increment that the TMA thread issues one item ahead and publishes to the other roles
// through a small ring in shared memory. Which CTA takes which item does not affect any
// result. Warp roles: warp 0 issues TMA loads (and L2 prefetches for the item after the
// current one), warp 1 issues MMAs and owns the TMEM allocation, warps 2..9 (two threads per
// TMEM lane) do the softmax arithmetic.
// Every mbarrier wait is bounded in time; on expiry the CTA records a status word and leaves.
#include "ec_common.cuh"

#include <cuda.h>
#include <type_traits>

namespace ec {

namespace {

constexpr int kTileRows = 128;            // rows of a tile = MMA M = MMA N
constexpr int kThreads = 320;             // 10 warps: TMA, MMA, 8 x softmax (two per TMEM lane quarter)
constexpr int kAccBufs = 2;               // TMEM accumulator buffers (128 columns each)
constexpr int kTmemCols = 256;
constexpr int kSched = 4;                 // slots of the ring that publishes item numbers to the roles
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

template <int D, int STAGES>
struct Smem {
    static constexpr int kTileBytes = kTileRows * D * 2;
    static constexpr int kStat = 0;
    static constexpr int kStage0 = kTileBytes;
    static constexpr int kLse = kStage0 + STAGES * kTileBytes;            // 2 x 128 floats
    static constexpr int kComb = kLse + kAccBufs * kTileRows * 4;         // 128 x float2: half-row results
    static constexpr int kBars = kComb + kTileRows * 8;
    // barrier slots (8 bytes each): stat_full, stat_empty, full[STAGES], empty[STAGES],
    // acc_full[2], acc_empty[2], lse_ready[2], comb_full, comb_empty, sched_full[kSched], sched_empty[kSched]
    static constexpr int kNumBars = 2 + 2 * STAGES + 3 * kAccBufs + 2 + 2 * kSched;
    static constexpr int kTmemSlot = kBars + kNumBars * 8;
    static constexpr int kAbort = kTmemSlot + 4;
    static constexpr int kSchedItems = (kAbort + 4 + 15) & ~15;           // kSched published items (int4 each)
    static constexpr int kTotal = kSchedItems + kSched * 16;
    static constexpr int kDynBytes = kTotal + 1024;                       // slack for 1024-byte alignment
};

// Geometry of the causal contraction with a visible prefix: query m sees keys n <= m + P.
struct Geometry {
    int Tq, P, ntq, ntk;
    __host__ __device__ int Tk() const { return Tq + P; }
    // pass 1: last key tile a query tile touches
    __host__ __device__ int jmax(int i) const { int j = (i * kTileRows + kTileRows - 1 + P) / kTileRows; return j < ntk - 1 ? j : ntk - 1; }
    // pass 2: first query tile that sees a key tile
    __host__ __device__ int imin(int j) const { int d = j * kTileRows - P; return d > 0 ? d / kTileRows : 0; }
};

// How the attention rows are folded into a per-key statistic (Sec. 3.2 "Importance Metrics").
// Query m enters pass 2 with weight 2^(wa + wb*(m - (Tq-1))): pass 1 stores lse minus that exponent,
// so the weight costs nothing per element. wa = wb = 0 is the plain sum; a moving average with
// factor beta is wa = log2(1-beta), wb = -log2(beta). Counting from the last query keeps the exponent
// small, hence exact to an fp32 ulp, for the newest queries, which are the ones whose weight matters
// (for a long prompt and a small beta the oldest queries' exponents reach tens of thousands, but
// their weights are zero to any precision). `mean` divides each key's total by the number of queries
// that can see it.
struct Fold {
    float wa, wb;
    int mean;
};

constexpr int kPass1 = 0, kPass2Sum = 1, kPass2Max = 2;

// MODE kPass1:    stationary = query tile i, streamed = key tiles jmax(i) .. 0      -> lse2 (and lse_out)
// MODE kPass2Sum: stationary = key tile j,   streamed = query tiles imin(j) .. ntq-1 -> scores (weighted sums)
// MODE kPass2Max: the same walk, keeping the maximum over the queries instead of the sum
// A streamed tile needs the mask only when 128*(i-j) + P < 127. lse2 is padded to ntq*128 entries
// per unit; entries past Tq hold +inf so that pass 2 gives those (non-existent) queries zero weight.
template <int D, int STAGES, int MODE>
__global__ void __launch_bounds__(kThreads, 2)
importance_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const Geometry geo, const Fold fold, int n_items, int tail_units, float c, float *__restrict__ lse2,
                  float *__restrict__ lse_out, float *__restrict__ scores, int *__restrict__ status,
                  int *__restrict__ next_item)
{
    constexpr bool PASS2 = MODE != kPass1;
    constexpr bool TAKE_MAX = MODE == kPass2Max;
    using L = Smem<D, STAGES>;
    constexpr int kTileBytes = L::kTileBytes;
    constexpr int kBoxes = D / 64;                          // TMA boxes (64 bf16 = 128 B wide) per tile
    constexpr int kBoxBytes = kTileRows * 128;
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((kTileRows >> 3) << 17) | ((kTileRows >> 4) << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + L::kBars;
    const uint32_t bar_stat_full = bars, bar_stat_empty = bars + 8u;
    auto bar_full = [&](int s) { return bars + 8u * (2 + s); };
    auto bar_empty = [&](int s) { return bars + 8u * (2 + STAGES + s); };
    auto bar_acc_full = [&](int b) { return bars + 8u * (2 + 2 * STAGES + b); };
    auto bar_acc_empty = [&](int b) { return bars + 8u * (2 + 2 * STAGES + kAccBufs + b); };
    auto bar_lse = [&](int b) { return bars + 8u * (2 + 2 * STAGES + 2 * kAccBufs + b); };
    const uint32_t bar_comb_full = bars + 8u * (2 + 2 * STAGES + 3 * kAccBufs);
    const uint32_t bar_comb_empty = bar_comb_full + 8u;
    auto bar_sched_full = [&](uint32_t k) { return bar_comb_empty + 8u * (1 + k); };
    auto bar_sched_empty = [&](uint32_t k) { return bar_comb_empty + 8u * (1 + kSched + k); };
    int4 *sched_s = reinterpret_cast<int4 *>(base_ptr + L::kSchedItems);   // {unit, stationary tile, first streamed tile, count}
    float2 *comb_s = reinterpret_cast<float2 *>(base_ptr + L::kComb);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(base_ptr + L::kTmemSlot);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(base_ptr + L::kAbort);
    float *lse_s = reinterpret_cast<float *>(base_ptr + L::kLse);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const CUtensorMap *map_stat = PASS2 ? &map_k : &map_q;
    const CUtensorMap *map_strm = PASS2 ? &map_q : &map_k;
    const int nts = PASS2 ? geo.ntk : geo.ntq;              // stationary tiles per unit
    const int grid_n = (int)gridDim.x;

    if (threadIdx.x == 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
    }
    // a CTA of this launch has already given up: leave at once instead of timing out again
    if (threadIdx.x == 0) *abort_flag = *reinterpret_cast<volatile int *>(status);
    __syncthreads();
    if (*abort_flag) return;

    if (threadIdx.x == 0) {
        mbar_init(bar_stat_full, 1);
        mbar_init(bar_stat_empty, 1);
        for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full(s), 1); mbar_init(bar_empty(s), 1); }
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(bar_acc_full(b), 1);
            mbar_init(bar_acc_empty(b), 8);
            mbar_init(bar_lse(b), 8 * 32);
        }
        mbar_init(bar_comb_full, 4 * 32);
        mbar_init(bar_comb_empty, 4 * 32);
        for (uint32_t k = 0; k < (uint32_t)kSched; ++k) {
            mbar_init(bar_sched_full(k), 1);
            mbar_init(bar_sched_empty(k), 1 + 8);           // the MMA thread and one lane of each softmax warp
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

    // Every role walks the same sequence of items with the same counters: `it` counts items
    // (stationary tiles), `tg` counts streamed tiles; ring slots and barrier phases derive from them.
    uint32_t it = 0, tg = 0;
    bool alive = true;

    // item -> unit, stationary tile, first streamed tile and number of streamed tiles. Units go in
    // order and a unit's items from the longest to the shortest, except for the last `tail_units`
    // units, which are taken together: all their longest items first, their shortest last. The work
    // handed out last is then made of short items of a few units (longest-first list scheduling),
    // and those units' tensors still fit the L2 together.
    const int n_units = n_items / nts, head_items = (n_units - tail_units) * nts;
    auto decode_item = [&](int item, int &unit, int &st, int &first, int &count) {
        int k;
        if (item < head_items) {
            unit = item / nts;
            k = item - unit * nts;
        } else {
            const int j = item - head_items;
            k = j / tail_units;
            unit = (n_units - tail_units) + (j - k * tail_units);
        }
        st = PASS2 ? k : nts - 1 - k;
        if (PASS2) { first = geo.imin(st); count = geo.ntq - first; }
        else       { first = geo.jmax(st); count = first + 1; }
    };
    auto stream_tile = [&](int first, int t) { return PASS2 ? first + t : first - t; };

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t armed = 0, stat_armed = 0;           // streamed tiles / stationary tiles whose copies were started
            int item = (int)blockIdx.x;                   // the first item needs no counter: one per CTA
            for (uint32_t k = 0; alive; ++k) {
                const uint32_t sl = k % kSched, sph = (k / kSched) & 1u;
                if (!mbar_wait(bar_sched_empty(sl), sph ^ 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                int unit = -1, st = 0, first = 0, count = 0;  // unit -1: no work left, every role leaves
                if (item < n_items) decode_item(item, unit, st, first, count);
                sched_s[sl] = make_int4(unit, st, first, count);
                mbar_arrive(bar_sched_full(sl));
                if (unit < 0) break;
                // the item after this one: asked for now, needed only when this item's copies are under way
                const int next = grid_n + atomicAdd(next_item, 1);
                // The item's first streamed tile goes out first: its ring stage was released by an
                // earlier MMA of the previous item, whereas the stationary buffer is free only once
                // that item's last MMA has completed.
                for (int t = 0; t < count; ++t, ++tg) {
                    const uint32_t s = tg % STAGES, ph = (tg / STAGES) & 1u;
                    if (!mbar_wait(bar_empty(s), ph ^ 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                    mbar_expect_tx(bar_full(s), kTileBytes);
#pragma unroll
                    for (int bx = 0; bx < kBoxes; ++bx)
                        tma_load_3d(base + L::kStage0 + s * kTileBytes + bx * kBoxBytes, map_strm, bx * 64,
                                    stream_tile(first, t) * kTileRows, unit, bar_full(s));
                    armed = tg + 1;
                    if (t == 0) {
                        if (!mbar_wait(bar_stat_empty, (it + 1u) & 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                        mbar_expect_tx(bar_stat_full, kTileBytes);
#pragma unroll
                        for (int bx = 0; bx < kBoxes; ++bx)
                            tma_load_3d(base + L::kStat + bx * kBoxBytes, map_stat, bx * 64, st * kTileRows, unit, bar_stat_full);
                        stat_armed = it + 1;
                    }
                }
                ++it;
                item = next;
            }
            if (*abort_flag) {
                // let copies that are still in flight land before the CTA gives its memory back
                if (stat_armed > 0) mbar_wait(bar_stat_full, (stat_armed - 1u) & 1u, abort_flag, status, 200000ull);
                for (uint32_t t = armed > (uint32_t)STAGES ? armed - STAGES : 0; t < armed; ++t)
                    mbar_wait(bar_full(t % STAGES), (t / STAGES) & 1u, abort_flag, status, 200000ull);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            for (uint32_t k = 0; alive; ++k) {
                const uint32_t sl = k % kSched, sph = (k / kSched) & 1u;
                if (!mbar_wait(bar_sched_full(sl), sph, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                const int4 d = sched_s[sl];
                mbar_arrive(bar_sched_empty(sl));
                if (d.x < 0) break;
                const int count = d.w;
                if (!mbar_wait(bar_stat_full, it & 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                for (int t = 0; t < count; ++t, ++tg) {
                    const uint32_t s = tg % STAGES, ph = (tg / STAGES) & 1u;
                    const uint32_t b = tg % kAccBufs, bph = (tg / kAccBufs) & 1u;
                    if (!mbar_wait(bar_acc_empty(b), bph ^ 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                    if (!mbar_wait(bar_full(s), ph, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t a0 = base + L::kStat, b0 = base + L::kStage0 + s * kTileBytes;
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint32_t off = (uint32_t)(kk / 4) * kBoxBytes + (uint32_t)(kk % 4) * 32u;
                        umma_bf16(tmem_base + b * kTileRows, umma_desc(a0 + off), umma_desc(b0 + off), kIdesc,
                                  kk > 0 ? 1u : 0u);
                    }
                    umma_commit(bar_empty(s));       // stage reusable once these MMAs have read it
                    umma_commit(bar_acc_full(b));    // accumulator ready for the softmax warps
                }
                if (alive) umma_commit(bar_stat_empty);   // stationary tile no longer read
                ++it;
            }
        }
    } else {
        // ---------------------------------------------------------------- softmax warps
        // Two warps share each TMEM lane quarter: warps 2..5 take columns 0..63 of a tile, warps
        // 6..9 columns 64..127. A row's two half results meet through shared memory at the end of
        // an item. Eight warps instead of four keep the ex2 pipe fed while others wait on TMEM.
        const int q4 = warp & 3;                              // TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;                     // which 64 columns of every tile
        const int r = q4 * 32 + lane;                         // row of the stationary tile = TMEM lane
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q4 * 32) << 16) + (uint32_t)(half * 64);
        const int Tk = geo.Tk();
        // The next item's description is normally picked up while this item's last tile is worked on
        // (the TMA thread publishes it ahead), and in pass 2 the load of its first lse entry starts
        // then, so that the start of an item costs no round trip to shared or global memory.
        int4 next_d = make_int4(-1, 0, 0, 0);
        float lse_next = 0.f;
        bool have_next = false;
        for (uint32_t k = 0; alive; ++k) {
            const uint32_t sl = k % kSched, sph = (k / kSched) & 1u;
            if (!have_next) {
                if (!mbar_wait(bar_sched_full(sl), sph, abort_flag, status)) { alive = false; break; }
                next_d = sched_s[sl];
            }
            const int unit = next_d.x, st = next_d.y, first = next_d.z, count = next_d.w;
            __syncwarp();                                         // every lane has read the slot
            if (lane == 0) mbar_arrive(bar_sched_empty(sl));
            if (unit < 0) break;
            const size_t lse_row = (size_t)unit * geo.ntq * kTileRows;
            float mrun = -INFINITY, Z = 0.f;                      // pass 1 running max / sum (log2 domain)
            float2 accA = make_float2(0.f, 0.f), accB = accA;     // pass 2 column sum, four chains
            float lse_ahead = 0.f;
            if (PASS2 && half == 0) lse_ahead = have_next ? lse_next : lse2[lse_row + (size_t)first * kTileRows + r];
            have_next = false;
            for (int t = 0; t < count; ++t, ++tg) {
                const uint32_t b = tg % kAccBufs, bph = (tg / kAccBufs) & 1u;
                const int tile = stream_tile(first, t);
                if (t == count - 1) {
                    // last tile: look (without waiting) whether the next item is published; the warp decides as one
                    const uint32_t nsl = (k + 1u) % kSched, nph = ((k + 1u) / kSched) & 1u;
                    have_next = __all_sync(0xffffffffu, mbar_try(bar_sched_full(nsl), nph));
                    if (have_next) next_d = sched_s[nsl];
                }
                // off = 128*(query tile - key tile) + P: element (row, col) is visible iff
                //   pass 1 (row = query, col = key):  col <= row + off
                //   pass 2 (row = key,  col = query): col >= row - off
                const int off = (PASS2 ? tile - st : st - tile) * kTileRows + geo.P;
                const bool masked = off < kTileRows - 1;
                if (PASS2) {
                    // the first-half threads stage one entry each of the tile's lse (fetched one tile
                    // ahead, so its latency hides behind the previous tile's math), then all wait
                    // (bounded) for the 128 entries. Every softmax thread, readers of the second half
                    // included, arrives on the tile's barrier: a thread that has passed the rendezvous
                    // of tile t+1 therefore knows that all 256 have finished reading tile t's entries,
                    // and only then may buffer b be overwritten for tile t+2.
                    if (half == 0) {
                        lse_s[b * kTileRows + r] = -lse_ahead;    // staged negated: exponent = v*c + (-lse)
                        mbar_arrive(bar_lse(b));
                        if (t + 1 < count)
                            lse_ahead = lse2[lse_row + (size_t)stream_tile(first, t + 1) * kTileRows + r];
                        else if (have_next && next_d.x >= 0)
                            lse_next = lse2[((size_t)next_d.x * geo.ntq + (size_t)next_d.z) * kTileRows + r];
                    } else {
                        mbar_arrive(bar_lse(b));
                    }
                    if (!mbar_wait(bar_lse(b), bph, abort_flag, status)) { alive = false; break; }
                }
                if (!mbar_wait(bar_acc_full(b), bph, abort_flag, status)) { alive = false; break; }
                tc_fence_after();

                // `ch` = index of the 32-column chunk inside the 128-column tile
                auto chunk = [&](uint32_t (&raw)[32], int ch, auto mask_tag) {
                    constexpr bool MASKED = decltype(mask_tag)::value;
                    float v[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(raw[i]);
                    if (!PASS2) {
                        if constexpr (MASKED) {
                            const int lim = r + off - ch * 32;            // columns i <= lim are visible
#pragma unroll
                            for (int i = 0; i < 32; ++i) if (i > lim) v[i] = -INFINITY;
                        }
                        float cm4[4] = {v[0], v[1], v[2], v[3]};      // four chains instead of one of 31
#pragma unroll
                        for (int i = 4; i < 32; ++i) cm4[i & 3] = fmaxf(cm4[i & 3], v[i]);
                        const float cm = fmaxf(fmaxf(cm4[0], cm4[1]), fmaxf(cm4[2], cm4[3]));
                        const float mnew = fmaxf(mrun, cm * c);
                        if (mnew != -INFINITY) {
                            float2 part[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                            sum_exp2(v, c, mnew, part);
                            Z = Z * fast_exp2(mrun - mnew) + ((part[0].x + part[0].y) + (part[1].x + part[1].y));
                            mrun = mnew;
                        }
                    } else {
                        const float4 *ls = reinterpret_cast<const float4 *>(lse_s + b * kTileRows + ch * 32);
                        const int lim = r - off - ch * 32;                // columns i >= lim are visible
                        const float2 c2 = make_float2(c, c);
#pragma unroll
                        for (int i4 = 0; i4 < 8; ++i4) {
                            const float4 nl = ls[i4];                     // -lse of four query rows
                            const float2 a01 = __ffma2_rn(make_float2(v[i4 * 4 + 0], v[i4 * 4 + 1]), c2, make_float2(nl.x, nl.y));
                            const float2 a23 = __ffma2_rn(make_float2(v[i4 * 4 + 2], v[i4 * 4 + 3]), c2, make_float2(nl.z, nl.w));
                            const float2 e01 = exp2_pair(a01, i4 * 2), e23 = exp2_pair(a23, i4 * 2 + 1);
                            float p0 = e01.x, p1 = e01.y, p2 = e23.x, p3 = e23.y;
                            if constexpr (MASKED) {
                                if (i4 * 4 + 0 < lim) p0 = 0.f;
                                if (i4 * 4 + 1 < lim) p1 = 0.f;
                                if (i4 * 4 + 2 < lim) p2 = 0.f;
                                if (i4 * 4 + 3 < lim) p3 = 0.f;
                            }
                            if constexpr (TAKE_MAX) {
                                accA.x = fmaxf(accA.x, p0); accA.y = fmaxf(accA.y, p1);
                                accB.x = fmaxf(accB.x, p2); accB.y = fmaxf(accB.y, p3);
                            } else {
                                accA = __fadd2_rn(accA, make_float2(p0, p1));
                                accB = __fadd2_rn(accB, make_float2(p2, p3));
                            }
                        }
                    }
                };

                // Only tiles the diagonal crosses pay for the mask: they run a separate instance.
                auto tile_body = [&](auto mask_tag) {
                    constexpr bool MASKED = decltype(mask_tag)::value;
                    const uint32_t col0 = lane_addr + b * kTileRows;
                    // A chunk the mask hides from all 32 rows of this warp is neither read nor
                    // exponentiated (on a diagonal tile that is 6 of the 16 warp x chunk blocks).
                    //   pass 1: column visible iff col <= row + off  -> hidden iff first col > last row + off
                    //   pass 2: column visible iff col >= row - off  -> hidden iff last col < first row - off
                    auto hidden = [&](int ch) {
                        if (!MASKED) return false;
                        return PASS2 ? (ch * 32 + 31 < q4 * 32 - off) : (ch * 32 > q4 * 32 + 31 + off);
                    };
                    const bool skip_a = hidden(half * 2), skip_b = hidden(half * 2 + 1);   // warp-uniform
                    auto release = [&]() {
                        tc_fence_before();               // all TMEM reads of this tile are done:
                        __syncwarp();                    // hand the accumulator back before the last chunk's math
                        if (lane == 0) mbar_arrive(bar_acc_empty(b));
                    };
                    if (!skip_a && !skip_b) {
                        // this thread's 64 columns: the second 32 are in flight while the first are processed
                        uint32_t ra[32], rb[32];
                        tmem_ld32_async(col0, ra);
                        tmem_ld_wait(ra);
                        tmem_ld32_async(col0 + 32, rb);
                        chunk(ra, half * 2, mask_tag);
                        tmem_ld_wait(rb);
                        release();
                        chunk(rb, half * 2 + 1, mask_tag);
                    } else if (skip_a && skip_b) {
                        release();
                    } else {
                        const int which = skip_a ? 1 : 0;     // the one chunk some row of the warp can see
                        uint32_t ra[32];
                        tmem_ld32_async(col0 + 32 * which, ra);
                        tmem_ld_wait(ra);
                        release();
                        chunk(ra, half * 2 + which, mask_tag);
                    }
                };
                if (masked) tile_body(std::true_type{});
                else tile_body(std::false_type{});
            }
            if (!alive) break;

            // the two halves of a row meet: the second-half thread hands its result over
            const uint32_t iph = it & 1u;
            const float own = TAKE_MAX ? fmaxf(fmaxf(accA.x, accA.y), fmaxf(accB.x, accB.y))
                                       : (accA.x + accA.y) + (accB.x + accB.y);
            if (half == 1) {
                if (!mbar_wait(bar_comb_empty, iph ^ 1u, abort_flag, status)) { alive = false; break; }
                comb_s[r] = PASS2 ? make_float2(own, 0.f) : make_float2(mrun, Z);
                mbar_arrive(bar_comb_full);
            } else {
                if (!mbar_wait(bar_comb_full, iph, abort_flag, status)) { alive = false; break; }
                const float2 o = comb_s[r];
                mbar_arrive(bar_comb_empty);
                const int row = st * kTileRows + r;
                if (!PASS2) {
                    const float M = fmaxf(mrun, o.x);             // finite: column 0 of some tile is visible
                    const float Zs = Z * fast_exp2(mrun - M) + o.y * fast_exp2(o.x - M);
                    const float l2 = (row < geo.Tq) ? M + __log2f(Zs) : INFINITY;
                    lse2[lse_row + row] = l2 - (fold.wa + fold.wb * (float)(row - (geo.Tq - 1)));   // +inf stays +inf
                    if (lse_out && row < geo.Tq) lse_out[(size_t)unit * geo.Tq + row] = l2 * kLn2;
                } else if (row < Tk) {
                    float total = TAKE_MAX ? fmaxf(own, o.x) : own + o.x;
                    if (fold.mean) total /= (float)(geo.Tq - (row > geo.P ? row - geo.P : 0));   // queries that see this key
                    scores[(size_t)unit * Tk + row] = total;
                }
            }
            ++it;
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
    const int unit = blockIdx.x;
    const int m = blockIdx.y * blockDim.x + threadIdx.x;
    if (m >= Tpad) return;
    lse2[(size_t)unit * Tpad + m] = (m < T) ? lse_nat[(size_t)unit * T + m] * kLog2e : INFINITY;
}

// One CTA waits, with the same bounded wait the importance kernels use, on a barrier that
// nothing ever completes: the wait has to expire, flag the status word and let the kernel end.
__global__ void wait_selftest_kernel(int *status, unsigned long long limit_ns)
{
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, &abort_flag, status, limit_ns);
}

int sm_count()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 148;
    return n;
}

template <int D, int STAGES>
cudaError_t launch_passes(const CUtensorMap &mq, const CUtensorMap &mk, int units, const Geometry &geo, const Fold &fold,
                          bool take_max, float c, float *lse2, float *lse_out, float *scores, int *status, bool first_pass,
                          cudaStream_t stream)
{
    constexpr int smem = Smem<D, STAGES>::kDynBytes;
    cudaError_t e = cudaFuncSetAttribute(importance_kernel<D, STAGES, kPass1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(importance_kernel<D, STAGES, kPass2Sum>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(importance_kernel<D, STAGES, kPass2Max>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    const long long resident = 2LL * sm_count();              // two persistent CTAs per SM
    const long long items1 = (long long)units * geo.ntq, items2 = (long long)units * geo.ntk;
    const unsigned grid1 = (unsigned)(items1 < resident ? items1 : resident);
    const unsigned grid2 = (unsigned)(items2 < resident ? items2 : resident);
    // units whose items are handed out longest-first at the end: about three items per CTA
    auto tail_of = [&](int nt) { const long long v = (3 * resident + nt - 1) / nt; return (int)(v < units ? v : units); };
    const int tail1 = tail_of(geo.ntq), tail2 = tail_of(geo.ntk);
    // the passes' item counters: words 1 and 2 of the status block, zeroed with it at the start of the call
    if (first_pass)
        importance_kernel<D, STAGES, kPass1><<<grid1, kThreads, smem, stream>>>(mq, mk, geo, fold, (int)items1, tail1, c, lse2,
                                                                              lse_out, scores, status, status + 1);
    if (take_max)
        importance_kernel<D, STAGES, kPass2Max><<<grid2, kThreads, smem, stream>>>(mq, mk, geo, fold, (int)items2, tail2, c, lse2,
                                                                                 lse_out, scores, status, status + 2);
    else
        importance_kernel<D, STAGES, kPass2Sum><<<grid2, kThreads, smem, stream>>>(mq, mk, geo, fold, (int)items2, tail2, c, lse2,
                                                                                 lse_out, scores, status, status + 2);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_wait_selftest(void *ws, unsigned limit_us, cudaStream_t stream)
{
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return e;
    wait_selftest_kernel<<<1, 32, 0, stream>>>(static_cast<int *>(ws), (unsigned long long)limit_us * 1000ull);
    return cudaGetLastError();
}

size_t importance_workspace_bytes(int N, int H, int T, int D)
{
    (void)D;
    const size_t nt = (size_t)(T + kTileRows - 1) / kTileRows;
    return kStatusBytes + (size_t)N * H * nt * kTileRows * sizeof(float);   // status block + padded lse
}

// lse_in == nullptr: both passes. Otherwise the caller's normaliser replaces pass 1 (plain sum only).
// Q: [units, Tq, D]; K: [units, P + Tq, D]; scores: [units, P + Tq]; lse_out / lse_in: [units, Tq].
// statistic: EC_STAT_*; beta in (0, 1) is read for the moving average only.
cudaError_t launch_importance(const void *Q, const void *K, float *scores, float *lse_out, const float *lse_in,
                              int N, int H, int Tq, int P, int D, float scale, int statistic, double beta, void *ws,
                              cudaStream_t stream)
{
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return e;
    int *status = static_cast<int *>(ws);
    float *lse2 = reinterpret_cast<float *>(static_cast<char *>(ws) + kStatusBytes);
    const int units = N * H;
    Geometry geo;
    geo.Tq = Tq;
    geo.P = P;
    geo.ntq = (Tq + kTileRows - 1) / kTileRows;
    geo.ntk = (Tq + P + kTileRows - 1) / kTileRows;
    if ((long long)units * geo.ntk > 0x7FFF0000LL) return cudaErrorInvalidConfiguration;   // item numbers (plus the grid size) stay in an int
    Fold fold = {0.f, 0.f, statistic == EC_STAT_MEAN ? 1 : 0};
    if (statistic == EC_STAT_MOVING_AVERAGE) {
        const double lb = log2(beta);
        fold.wa = (float)log2(1.0 - beta);
        fold.wb = (float)(-lb);
    }
    CUtensorMap mq, mk;
    if (!make_map(&mq, Q, units, Tq, D) || !make_map(&mk, K, units, Tq + P, D)) return cudaErrorInvalidValue;
    if (lse_in) {
        dim3 g(units, (geo.ntq * kTileRows + 255) / 256);
        lse_import_kernel<<<g, 256, 0, stream>>>(lse_in, lse2, Tq, geo.ntq * kTileRows);
    }
    const float c = scale * kLog2e;
    const bool take_max = statistic == EC_STAT_MAX;
    if (D == 128)
        return launch_passes<128, 2>(mq, mk, units, geo, fold, take_max, c, lse2, lse_out, scores, status,
                                     lse_in == nullptr, stream);
    return launch_passes<64, 4>(mq, mk, units, geo, fold, take_max, c, lse2, lse_out, scores, status, lse_in == nullptr,
                                stream);
}

}  // namespace ec
