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
// result. Warp roles: warp 0 issues TMA loads, warp 1 issues MMAs and owns the TMEM allocation, warps 2..9 (two threads per
// TMEM lane) do the softmax arithmetic.
// Every mbarrier wait is bounded in time; on expiry the CTA records a status word and leaves.
#include "ec_tc.cuh"

#include <type_traits>

namespace ec {

namespace {

constexpr int kThreads = 320;             // 10 warps: TMA, MMA, 8 x softmax (two per TMEM lane quarter)
constexpr int kAccBufs = 2;               // TMEM accumulator buffers (128 columns each)
constexpr int kTmemCols = 256;
constexpr int kSched = 4;                 // slots of the ring that publishes item numbers to the roles
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
    // The kernel behind this one on the stream (pass 2 behind pass 1, the selection behind pass 2) may be
    // scheduled as soon as CTAs of this one leave; it waits for this grid to finish before it reads anything.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // Pass 2 is launched with programmatic stream serialization: its CTAs take the places pass-1 CTAs
    // free and wait here, so the launch latency falls under pass 1's tail. (A no-op otherwise.)
    if (PASS2) asm volatile("griddepcontrol.wait;" ::: "memory");
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
    cudaError_t e1 = cudaGetLastError();
    if (e1 != cudaSuccess) return e1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid2);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int n2 = (int)items2;
    int *counter2 = status + 2;
    if (take_max)
        return cudaLaunchKernelEx(&cfg, importance_kernel<D, STAGES, kPass2Max>, mq, mk, geo, fold, n2, tail2, c, lse2, lse_out,
                                  scores, status, counter2);
    return cudaLaunchKernelEx(&cfg, importance_kernel<D, STAGES, kPass2Sum>, mq, mk, geo, fold, n2, tail2, c, lse2, lse_out,
                              scores, status, counter2);
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
// lse_in == kLseInWorkspace: the padded log2-domain normaliser is already in the workspace (left there
// by the prefill attention kernel, whose launch also zeroed the status block): column-sum pass only.
// Q: [units, Tq, D]; K: [units, P + Tq, D]; scores: [units, P + Tq]; lse_out / lse_in: [units, Tq].
// statistic: EC_STAT_*; beta in (0, 1) is read for the moving average only.
cudaError_t launch_importance(const void *Q, const void *K, float *scores, float *lse_out, const float *lse_in,
                              int N, int H, int Tq, int P, int D, float scale, int statistic, double beta, void *ws,
                              cudaStream_t stream)
{
    const bool in_ws = lse_in == kLseInWorkspace;
    if (!in_ws) {
        cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, stream);
        if (e != cudaSuccess) return e;
    }
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
    if (lse_in && !in_ws) {
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
