// Decode attention over the compacted cache plus the step's new row, with the new row
// written into the slot freed by fixed-point elimination (Sec. 3.3 "Output Generation").
// HBM-bound: every cached K and V row is read once per step with 16-byte loads, so the
// kernel is built to spend as few instructions per byte as possible:
//  - LPR = D/8 lanes share a row (8 bf16 each); a lane group takes blocks of 8 consecutive
//    rows, so 16 independent 16-byte loads per lane are in flight;
//  - the 8 partial dot products of a block are reduced across the group with a transposing
//    butterfly (7 shuffles instead of 8 x log2(LPR)), which leaves each row's score on one lane
//    (pair), so the exponential is evaluated once per row, not once per lane;
//  - multiply-adds are issued as packed fp32 pairs (__ffma2_rn).
#include "ec_common.cuh"

namespace ec {

namespace {

// Threads per CTA. Small CTAs let at least 7 be resident per SM, so that the 1024 units of a
// 7B-shaped single-sequence step (6.9 per SM) run as one balanced wave.
#ifndef EC_DEC_THREADS
#define EC_DEC_THREADS 64
#endif
#ifndef EC_DEC_MIN_CTAS
#define EC_DEC_MIN_CTAS 8
#endif
constexpr int kDecThreads = EC_DEC_THREADS;
#ifndef EC_DEC_TARGET
#define EC_DEC_TARGET (148 * 4)
#endif
constexpr int kMaxSplits = EC_DEC_TARGET;     // CTAs aimed at when there are fewer units than that; also the most splits a unit gets
#ifndef EC_DEC_MIN_ROWS
#define EC_DEC_MIN_ROWS 256
#endif
constexpr int kMinRowsPerSplit = EC_DEC_MIN_ROWS;
constexpr int kBlk = 8;                       // rows per block of a lane group

// The cache is written later in the same kernel, so no read-only (.nc) path here.
__device__ __forceinline__ uint4 ld_row(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Same load served from L2: used for the rows read after waiting for the previous step, so that a
// line which an earlier read of a neighbouring row may have left in L1 cannot be served stale.
__device__ __forceinline__ uint4 ld_row_l2(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float2 unpack2(uint32_t w) { return make_float2(bf16lo(w), bf16hi(w)); }

// Partial dot product of this lane's 8 elements (q pre-multiplied by scale*log2e).
__device__ __forceinline__ float dot8(const float2 (&q2)[4], const uint4 &k)
{
    float2 d = __ffma2_rn(q2[0], unpack2(k.x), make_float2(0.f, 0.f));
    d = __ffma2_rn(q2[1], unpack2(k.y), d);
    d = __ffma2_rn(q2[2], unpack2(k.z), d);
    d = __ffma2_rn(q2[3], unpack2(k.w), d);
    return d.x + d.y;
}

__device__ __forceinline__ void axpy8(float2 (&acc)[4], float p, const uint4 &v)
{
    const float2 p2 = make_float2(p, p);
    acc[0] = __ffma2_rn(p2, unpack2(v.x), acc[0]);
    acc[1] = __ffma2_rn(p2, unpack2(v.y), acc[1]);
    acc[2] = __ffma2_rn(p2, unpack2(v.z), acc[2]);
    acc[3] = __ffma2_rn(p2, unpack2(v.w), acc[3]);
}

// Running softmax state of a lane group, log2 domain. `lsum` is a per-lane partial: each
// row's weight is added on the lanes that own the row (LPR/8 of them).
struct GroupState {
    float m, lsum;
    float2 acc[4];
};

// One block of up to 8 consecutive cache rows starting at `row`. GUARD: rows >= row_end are
// skipped (their loads are clamped to the last valid row and their score is -inf).
// FRESH: the block is read after the wait for the previous step and must not come from L1.
template <int LPR, bool GUARD, bool FRESH = false>
__device__ __forceinline__ void process_block(GroupState &st, const float2 (&q2)[4], const uint4 *Kl, const uint4 *Vl,
                                              int row, int row_end, int l, unsigned gmask)
{
    uint4 rk[kBlk], rv[kBlk];
#pragma unroll
    for (int r = 0; r < kBlk; ++r) {
        const int j = GUARD ? min(row + r, row_end - 1) : row + r;
        rk[r] = FRESH ? ld_row_l2(Kl + (size_t)j * LPR) : ld_row(Kl + (size_t)j * LPR);
    }
#pragma unroll
    for (int r = 0; r < kBlk; ++r) {
        const int j = GUARD ? min(row + r, row_end - 1) : row + r;
        rv[r] = FRESH ? ld_row_l2(Vl + (size_t)j * LPR) : ld_row(Vl + (size_t)j * LPR);
    }
    float s[kBlk];
#pragma unroll
    for (int r = 0; r < kBlk; ++r) s[r] = dot8(q2, rk[r]);

    // transposing butterfly: after the three steps lane l holds the sum for row (l * 8 / LPR)
#pragma unroll
    for (int step = 0; step < 3; ++step) {
        const int o = LPR >> (step + 1);
        const int n = kBlk >> step;                 // values held before this step
        const bool upper = (l & o) != 0;
#pragma unroll
        for (int i = 0; i < n / 2; ++i) {
            const float keep = upper ? s[i + n / 2] : s[i];
            const float send = upper ? s[i] : s[i + n / 2];
            s[i] = keep + __shfl_xor_sync(gmask, send, o);
        }
    }
    float sc = s[0];
    if (LPR == 16) sc += __shfl_xor_sync(gmask, sc, 1);
    if (GUARD) {
        const int my_row = row + l * kBlk / LPR;
        if (my_row >= row_end) sc = -INFINITY;
    }
    float bm = sc;
#pragma unroll
    for (int o = LPR / 2; o >= LPR / 8; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(gmask, bm, o));
    const float mn = fmaxf(st.m, bm);               // finite: a block always has a valid first row
    const float corr = fast_exp2(st.m - mn);        // first block: exp2(-inf) = 0
    const float p = fast_exp2(sc - mn);
    st.m = mn;
    st.lsum = fmaf(st.lsum, corr, p);
    const float2 c2 = make_float2(corr, corr), z2 = make_float2(0.f, 0.f);
#pragma unroll
    for (int i = 0; i < 4; ++i) st.acc[i] = __ffma2_rn(st.acc[i], c2, z2);
#pragma unroll
    for (int r = 0; r < kBlk; ++r) {
        const float pr = __shfl_sync(gmask, p, r * LPR / kBlk, LPR);
        axpy8(st.acc, pr, rv[r]);
    }
}

// grid.x = units * splits. Rows 0..len-1 come from the cache, row `len` is the new token.
// splits == 1: writes out (bf16) and stores the new row into `write_slot`.
// splits  > 1: every CTA writes (acc[D], max, sum) of its rows to `partials` and counts itself in
// `counters[unit]`; the CTA that arrives last (nobody waits for anybody) merges the unit's partials,
// writes out, stores the new row and puts the counter back to zero for the next launch.
// THREADS = 64 is the shape for launches that fill the GPU. When a launch has too few CTAs for that (a
// single layer's units), wider CTAs give a unit more lane groups, so that a group walks one or two blocks
// of rows instead of four or five one after the other: the step is then a shorter chain of memory round trips.
template <int LPR, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == kDecThreads ? EC_DEC_MIN_CTAS : 1)
decode_kernel(const uint4 *__restrict__ q, const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new,
              uint4 *Kc, uint4 *Vc, int cap, int len, int write_slot, int defer_from, float scale_log2e,
              __nv_bfloat16 *__restrict__ out, float *partials, int *counters, int splits, int release_early)
{
    constexpr int D = LPR * 8;
    constexpr int G = THREADS / LPR;
    __shared__ float sm_acc[G][D];
    __shared__ float sm_m[G], sm_l[G];
    __shared__ int sm_last;
    __shared__ float sm_pm[kMaxSplits], sm_pl[kMaxSplits];   // (max, sum) of every split of the unit

    // Launched with programmatic stream serialization. defer_from < 0: nothing in global memory
    // is touched before the previous kernel of the stream has completed. defer_from >= 0: the
    // kernels in front are earlier decode steps of the same call, and none of them writes a cache
    // row below `defer_from` (new rows only ever go to the slots of the most recent rows or are
    // appended). Those stable rows are read at once, however many earlier steps are still in
    // flight, and the next step is released before anything else, so that its launch latency and
    // its reading hide behind this step; the rows from `defer_from` on, and every write, wait for
    // the predecessor to complete (and with it all steps before it).
    if (defer_from < 0) grid_dependency_wait();
    if (defer_from < 0 || release_early) grid_launch_dependents();

    const int unit = blockIdx.x / splits;
    const int split = blockIdx.x - unit * splits;
    const int g = threadIdx.x / LPR;
    const int l = threadIdx.x - g * LPR;
    const unsigned gmask = ((LPR == 16) ? 0xFFFFu : 0xFFu) << ((threadIdx.x & 31) / LPR * LPR);

    uint4 *Kcu = Kc + (size_t)unit * cap * LPR;
    uint4 *Vcu = Vc + (size_t)unit * cap * LPR;
    const uint4 *knu = k_new + (size_t)unit * LPR;
    const uint4 *vnu = v_new + (size_t)unit * LPR;

    float2 q2[4];
    {
        const uint4 qv = q[(size_t)unit * LPR + l];
        const float2 s2 = make_float2(scale_log2e, scale_log2e), z2 = make_float2(0.f, 0.f);
        q2[0] = __ffma2_rn(unpack2(qv.x), s2, z2);
        q2[1] = __ffma2_rn(unpack2(qv.y), s2, z2);
        q2[2] = __ffma2_rn(unpack2(qv.z), s2, z2);
        q2[3] = __ffma2_rn(unpack2(qv.w), s2, z2);
    }

    // cached rows of this split: [r0, r1); the last split also takes the new row
    const int per = (len + splits - 1) / splits;
    const int r0 = min(split * per, len), r1 = min(r0 + per, len);
    const int nfull = (r1 - r0) / kBlk;

    GroupState st;
    st.m = -INFINITY;
    st.lsum = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) st.acc[i] = make_float2(0.f, 0.f);

    const uint4 *Kl = Kcu + l, *Vl = Vcu + l;
    const bool has_tail = r0 + nfull * kBlk < r1;
    if (defer_from < 0) {
        for (int b = g; b < nfull; b += G) process_block<LPR, false>(st, q2, Kl, Vl, r0 + b * kBlk, r1, l, gmask);
        if (has_tail && (nfull % G) == g) process_block<LPR, true>(st, q2, Kl, Vl, r0 + nfull * kBlk, r1, l, gmask);
    } else {
        // whole blocks of stable rows first; the rest after the predecessor has completed
        const int early = (min(max(defer_from, r0), r1) - r0) / kBlk;
        for (int b = g; b < early; b += G) process_block<LPR, false>(st, q2, Kl, Vl, r0 + b * kBlk, r1, l, gmask);
        grid_dependency_wait();
        if (!release_early) grid_launch_dependents();
        for (int b = early + (g - early % G + G) % G; b < nfull; b += G)     // block b stays with group b % G
            process_block<LPR, false, true>(st, q2, Kl, Vl, r0 + b * kBlk, r1, l, gmask);
        if (has_tail && (nfull % G) == g) process_block<LPR, true, true>(st, q2, Kl, Vl, r0 + nfull * kBlk, r1, l, gmask);
    }

    // per-lane partial sums -> group sum (rows are owned by LPR/8 lanes each)
    float lsum = st.lsum;
#pragma unroll
    for (int o = LPR / 2; o >= 1; o >>= 1) lsum += __shfl_xor_sync(gmask, lsum, o);
    lsum *= (float)kBlk / (float)LPR;

    if (split == splits - 1 && g == G - 1) {
        // the step's own (k_new, v_new) row, straight from the inputs
        const uint4 kn = ld_row(knu + l), vn = ld_row(vnu + l);
        float sc = dot8(q2, kn);
#pragma unroll
        for (int o = LPR / 2; o >= 1; o >>= 1) sc += __shfl_xor_sync(gmask, sc, o);
        const float mn = fmaxf(st.m, sc);
        const float corr = fast_exp2(st.m - mn), p = fast_exp2(sc - mn);
        st.m = mn;
        lsum = fmaf(lsum, corr, p);
        const float2 c2 = make_float2(corr, corr), z2 = make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < 4; ++i) st.acc[i] = __ffma2_rn(st.acc[i], c2, z2);
        axpy8(st.acc, p, vn);
    }

    if (l == 0) { sm_m[g] = st.m; sm_l[g] = lsum; }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        sm_acc[g][l * 8 + 2 * i] = st.acc[i].x;
        sm_acc[g][l * 8 + 2 * i + 1] = st.acc[i].y;
    }
    __syncthreads();   // also orders every cache read of this CTA before the slot write below

    for (int d = threadIdx.x; d < D; d += THREADS) {
        float M = -INFINITY;
#pragma unroll
        for (int gg = 0; gg < G; ++gg) M = fmaxf(M, sm_m[gg]);
        float L = 0.f, A = 0.f;
#pragma unroll
        for (int gg = 0; gg < G; ++gg) {
            const float mg = sm_m[gg];
            const float w = (mg == -INFINITY) ? 0.f : fast_exp2(mg - M);
            L = fmaf(sm_l[gg], w, L);
            A = fmaf(sm_acc[gg][d], w, A);
        }
        if (splits == 1) {
            out[(size_t)unit * D + d] = __float2bfloat16_rn(A / L);
        } else {
            float *p = partials + (size_t)blockIdx.x * (D + 2);
            p[d] = A;
            if (d == 0) { p[D] = M; p[D + 1] = L; }
        }
    }
    bool finish = splits == 1;
    if (splits > 1) {
        // last arriver of the unit: its own partial and, through the fences, everybody else's are visible
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) sm_last = (atomicAdd(counters + unit, 1) == splits - 1);
        __syncthreads();
        finish = sm_last != 0;
        if (finish) {
            __threadfence();
            if (threadIdx.x == 0) counters[unit] = 0;
            // the splits' (max, sum) pairs first, all loads in flight at once, then their weights
            const float *p = partials + (size_t)unit * splits * (D + 2);
            for (int sp = threadIdx.x; sp < splits; sp += THREADS) {
                sm_pm[sp] = __ldcg(p + (size_t)sp * (D + 2) + D);
                sm_pl[sp] = __ldcg(p + (size_t)sp * (D + 2) + D + 1);
            }
            __syncthreads();
            float M = -INFINITY;
            for (int sp = 0; sp < splits; ++sp) M = fmaxf(M, sm_pm[sp]);
            float L = 0.f;
            for (int sp = 0; sp < splits; ++sp) {
                const float ms = sm_pm[sp];
                L = fmaf(sm_pl[sp], (ms == -INFINITY) ? 0.f : fast_exp2(ms - M), L);
            }
            const float inv_l = 1.f / L;
            for (int d = threadIdx.x; d < D; d += THREADS) {
                float A = 0.f;
#pragma unroll 4
                for (int sp = 0; sp < splits; ++sp) {
                    const float ms = sm_pm[sp];
                    A = fmaf(__ldcg(p + (size_t)sp * (D + 2) + d), (ms == -INFINITY) ? 0.f : fast_exp2(ms - M), A);
                }
                out[(size_t)unit * D + d] = __float2bfloat16_rn(A * inv_l);
            }
        }
    }
    // the new row takes the freed slot once every CTA of the unit has read its rows
    if (finish && threadIdx.x >= THREADS - 2 * LPR) {
        const int i = threadIdx.x - (THREADS - 2 * LPR);
        if (i < LPR) Kcu[(size_t)write_slot * LPR + i] = knu[i];
        else         Vcu[(size_t)write_slot * LPR + (i - LPR)] = vnu[i - LPR];
    }
}

}  // namespace

// Split the rows of a unit over several CTAs only when there are too few units to fill the GPU,
// and never into parts of fewer than 256 rows: a part has to stream for longer than the arrival
// counting and the merge of the partial results cost (measured per step with 64-row parts / 256-row
// parts: 32 units x 320 rows 5.8 / 5.2 us, 32 x 820 7.1 / 5.0, 40 x 1024 8.9 / 5.8, 8 x 128 4.7 / 2.2;
// 512-row parts are slower again).
int decode_splits(int units, int rows)
{
    const int target = kMaxSplits;
    if (units < 1) units = 1;
    int s = (target + units - 1) / units;
    int max_s = (rows + kMinRowsPerSplit - 1) / kMinRowsPerSplit;
    if (s > max_s) s = max_s;
    if (s < 1) s = 1;
    return s;
}

// Kernel launch that allows the launch latency of consecutive decode steps to overlap
// (the kernels themselves wait for their predecessor before touching memory).
template <typename... KArgs, typename... Args>
cudaError_t launch_overlapped(void (*kernel)(KArgs...), unsigned grid, unsigned block, cudaStream_t stream, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

int sm_count_cached()
{
    static int n = 0;
    if (n < 1) {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0)
            n = v;
        else
            return 148;
    }
    return n;
}

template <int LPR>
cudaError_t launch_decode_t(const void *q, const void *k_new, const void *v_new, void *Kc, void *Vc, int units,
                            int cap, int len, int write_slot, int defer_from, float sl2, void *out, float *partials,
                            int *counters, int splits, cudaStream_t stream)
{
#ifndef EC_DEC_EARLY_MIN_MB
#define EC_DEC_EARLY_MIN_MB 24
#endif
    const int release_early = (double)units * len * LPR * 32.0 >= EC_DEC_EARLY_MIN_MB * 1.0e6;   // K and V bytes of a step
    // the widest CTA with which the whole launch is still resident at once (about 512 threads per SM at this
    // kernel's register count)
    #ifndef EC_DEC_WIDE_X2
#define EC_DEC_WIDE_X2 2      // twice the factor by which a wide launch may exceed what is resident at once
#endif
    const long long ctas = (long long)units * splits, resident_threads = 512LL * sm_count_cached() * EC_DEC_WIDE_X2 / 2;
    auto go = [&](auto kernel, unsigned threads) {
        return launch_overlapped(kernel, (unsigned)ctas, threads, stream, (const uint4 *)q, (const uint4 *)k_new,
                                 (const uint4 *)v_new, (uint4 *)Kc, (uint4 *)Vc, cap, len, write_slot, defer_from, sl2,
                                 (__nv_bfloat16 *)out, partials, counters, splits, release_early);
    };
    if (ctas * 256 <= resident_threads) return go(decode_kernel<LPR, 256>, 256u);
    if (ctas * 128 <= resident_threads) return go(decode_kernel<LPR, 128>, 128u);
    return go(decode_kernel<LPR, kDecThreads>, (unsigned)kDecThreads);
}

cudaError_t launch_decode(const void *q, const void *k_new, const void *v_new, void *Kc, void *Vc,
                          int units, int D, int cap, int len, int write_slot, int defer_from, float scale, void *out,
                          float *partials, int *counters, int splits, cudaStream_t stream)
{
    const float sl2 = scale * 1.4426950408889634f;
    if ((long long)units * splits > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    if (D == 128)
        return launch_decode_t<16>(q, k_new, v_new, Kc, Vc, units, cap, len, write_slot, defer_from, sl2, out, partials,
                                   counters, splits, stream);
    return launch_decode_t<8>(q, k_new, v_new, Kc, Vc, units, cap, len, write_slot, defer_from, sl2, out, partials, counters,
                              splits, stream);
}

}  // namespace ec
