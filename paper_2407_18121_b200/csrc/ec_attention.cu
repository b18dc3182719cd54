// Causal attention of the prompt tokens that also hands out each row's softmax normaliser
// (the forward pass Algorithm 1 takes its attention from, Alg. 1 "Input"): with the normaliser
// known, the importance of Eq. 1 costs one more contraction (the column-sum pass) instead of two.
//   out[m] = sum_{n <= m+P} softmax_n(scale*<q_m,k_n>) * v_n        lse[m] = log sum_{n <= m+P} exp(scale*<q_m,k_n>)
//
// One CTA per SM works on two adjacent 128-row query tiles of one unit at a time (a work item),
// each served by its own team of eight softmax warps; the key and value tiles stream once for
// both, from tile 0 up to the upper tile's diagonal (the lower tile's team stops one tile earlier
// and normalises and stores its rows while the other team works on its diagonal tile). Per key
// tile and team:
//   S = Q K^T            tcgen05.mma, both operands K-major from TMA-staged shared memory, S in TMEM
//   P = 2^(c*S - m)      the team reads S (one row per thread pair), writes P as bf16 over the
//                        first half of S's own TMEM columns
//   O += P V             tcgen05.mma with P as the TMEM operand and the V tile as an MN-major
//                        shared-memory operand (rows of V are contiguous along the head dimension)
// The tensor cores execute in issue order, and the issuing thread alternates between the teams
// (P V of team A, next S of team A, P V of team B, next S of team B), so one team's products run
// under the other team's softmax. The running maximum m is only raised when a tile exceeds it by
// more than 8 (log2 domain), so the accumulator in TMEM is rescaled rarely: P never exceeds 2^8 and
// the result does not depend on when m is raised. The two threads of a row (64 columns of S each)
// agree on a tile's maximum through shared memory before either scales anything.
// (Measured alternatives: one query tile per CTA with P through shared memory was 10% slower at
// long prompts; splitting a key tile into two 64-key halves with their own S buffers, so that a
// team never waits for its own products, was 27% slower: the per-half handshakes cost more than
// the waits they remove.)
// Roles: warp 0 TMA, warp 1 MMA issue + TMEM allocation, warps 2..9 team 0 (upper tile), warps
// 10..17 team 1 (the tile below it; idle for the single tile left over when a unit has an odd
// number of tiles). Items are handed out as in the importance kernels (a counter, longest first
// inside a unit and over the last units). Every mbarrier wait is bounded in time; on expiry the CTA
// records a status word and leaves.
#include "ec_tc.cuh"

namespace ec {

namespace {

constexpr int kAttnThreads = 576;         // TMA, MMA, 2 teams x 8 softmax warps
constexpr int kAttnSched = 4;
constexpr int kAttnTmemCols = 512;        // S of both teams (2 x 128 columns), O of both teams (2 x up to 128)
constexpr float kRaiseBy = 8.f;           // the running maximum moves only when a tile exceeds it by this much

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
                 "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
                   "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
                   "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
                   "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
                 : "memory");
}

// 32 bytes in one store: a thread's rows are 256 bytes apart, so every store instruction of a warp touches
// 32 lines whatever its width; wider stores mean fewer of them.
__device__ __forceinline__ void st_global_32B(void *p, const uint4 &a, const uint4 &b)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}

__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// MN-major shared-memory operand with the 128-byte swizzle: 64 contiguous elements of the MN
// dimension per 128-byte row, 8 rows (steps of the contraction index) per 1024-byte group; `lbo`
// bytes to the next 64 elements of the MN dimension, `sbo` bytes to the next 8 steps of the
// contraction index.
__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t smem_addr, uint32_t lbo, uint32_t sbo)
{
    return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}

// D = A * B with A (bf16, one row per TMEM lane, two elements of the contraction index per 32-bit
// column) read from TMEM and B from shared memory; M = 128, K = 16.
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

template <int D>
struct AttnSmem {
    static constexpr int kTile = kTileRows * D * 2;                       // a Q, K or V tile
    static constexpr int kQ0 = 0;                                         // Q of team 0, team 1
    static constexpr int kK0 = 2 * kTile;                                 // two stages of K
    static constexpr int kV0 = kK0 + 2 * kTile;                           // two stages of V
    static constexpr int kExch = kV0 + 2 * kTile;                         // [2 teams][2 halves][128] row maxima of a tile
    static constexpr int kLsum = kExch + 2 * 2 * kTileRows * 4;           // [2 teams][2 halves][128] row sums of an item
    static constexpr int kBars = kLsum + 2 * 2 * kTileRows * 4;
    // q_full, q_empty, k_full[2], k_empty[2], v_full[2], v_empty[2], then per team: s_full, x_rdv, p_full,
    // pv_done, o_free, l_rdv; then sched_full[4], sched_empty[4]
    static constexpr int kNumBars = 2 + 4 + 4 + 2 * 6 + 2 * kAttnSched;
    static constexpr int kTmemSlot = kBars + kNumBars * 8;
    static constexpr int kAbort = kTmemSlot + 4;
    static constexpr int kSchedItems = (kAbort + 4 + 15) & ~15;
    static constexpr int kTotal = kSchedItems + kAttnSched * 16;
    static constexpr int kDynBytes = kTotal + 1024;
};

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 1)
attention_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                 const __grid_constant__ CUtensorMap map_v, const Geometry geo, int n_items, int tail_units, float c,
                 __nv_bfloat16 *__restrict__ out, float *__restrict__ lse2, float *__restrict__ lse_out,
                 int *__restrict__ status, int *__restrict__ next_item)
{
    using L = AttnSmem<D>;
    constexpr int kTile = L::kTile;
    constexpr int kBoxes = D / 64;
    constexpr int kBoxBytes = kTileRows * 128;
    // S = Q K^T: M = 128 queries, N = 128 keys, both K-major
    constexpr uint32_t kIdescS = (1u << 4) | (1u << 7) | (1u << 10) | ((kTileRows >> 3) << 17) | ((kTileRows >> 4) << 24);
    // O += P V: M = 128 queries, N = D, A (P) from TMEM, B (V) MN-major
    constexpr uint32_t kIdescO = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((D >> 3) << 17) | ((kTileRows >> 4) << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + L::kBars;
    const uint32_t bar_q_full = bars, bar_q_empty = bars + 8u;
    auto bar_k_full = [&](uint32_t s) { return bars + 8u * (2 + s); };
    auto bar_k_empty = [&](uint32_t s) { return bars + 8u * (4 + s); };
    auto bar_v_full = [&](uint32_t s) { return bars + 8u * (6 + s); };
    auto bar_v_empty = [&](uint32_t s) { return bars + 8u * (8 + s); };
    // per team x: S ready, row maxima exchanged, P written, P V of the item's last tile done, O read out, row sums exchanged
    auto bar_s_full = [&](uint32_t x) { return bars + 8u * (10 + 6 * x); };
    auto bar_x_rdv = [&](uint32_t x) { return bars + 8u * (11 + 6 * x); };
    auto bar_p_full = [&](uint32_t x) { return bars + 8u * (12 + 6 * x); };
    auto bar_pv_done = [&](uint32_t x) { return bars + 8u * (13 + 6 * x); };
    auto bar_o_free = [&](uint32_t x) { return bars + 8u * (14 + 6 * x); };
    auto bar_l_rdv = [&](uint32_t x) { return bars + 8u * (15 + 6 * x); };
    auto bar_sched_full = [&](uint32_t k) { return bars + 8u * (22 + k); };
    auto bar_sched_empty = [&](uint32_t k) { return bars + 8u * (22 + kAttnSched + k); };
    float *exch_s = reinterpret_cast<float *>(base_ptr + L::kExch);
    float *lsum_s = reinterpret_cast<float *>(base_ptr + L::kLsum);
    int4 *sched_s = reinterpret_cast<int4 *>(base_ptr + L::kSchedItems);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(base_ptr + L::kTmemSlot);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(base_ptr + L::kAbort);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nps = (geo.ntq + 1) / 2;                     // items (tile pairs) per unit
    const int grid_n = (int)gridDim.x;

    if (threadIdx.x == 32) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_q) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    }
    // the column-sum pass that may follow is launched with programmatic stream serialization: it may be
    // scheduled as CTAs of this grid leave, and waits for the whole grid before it reads the normaliser
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) *abort_flag = *reinterpret_cast<volatile int *>(status);
    __syncthreads();
    if (*abort_flag) return;

    if (threadIdx.x == 0) {
        mbar_init(bar_q_full, 1);
        mbar_init(bar_q_empty, 1);
        for (uint32_t s = 0; s < 2; ++s) {
            mbar_init(bar_k_full(s), 1); mbar_init(bar_k_empty(s), 1);
            mbar_init(bar_v_full(s), 1); mbar_init(bar_v_empty(s), 1);
        }
        for (uint32_t x = 0; x < 2; ++x) {
            mbar_init(bar_s_full(x), 1);
            mbar_init(bar_x_rdv(x), 8 * 32);
            mbar_init(bar_p_full(x), 8 * 32);
            mbar_init(bar_pv_done(x), 1);
            mbar_init(bar_o_free(x), 8);
            mbar_init(bar_l_rdv(x), 8 * 32);
        }
        for (uint32_t k = 0; k < (uint32_t)kAttnSched; ++k) {
            mbar_init(bar_sched_full(k), 1);
            mbar_init(bar_sched_empty(k), 1 + 16);          // the MMA thread and one lane of each softmax warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + (uint32_t)L::kTmemSlot), "r"((uint32_t)kAttnTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    auto tmem_s = [&](uint32_t x) { return tmem_base + x * (uint32_t)kTileRows; };               // S (and P over its first half)
    auto tmem_o = [&](uint32_t x) { return tmem_base + 2u * kTileRows + x * (uint32_t)kTileRows; };

    // item -> unit, upper query tile (team 0), its highest key tile and number of key tiles (streamed
    // in ascending order). Team 1 takes the tile below (if there is one) and its own, smaller number.
    const int n_units = n_items / nps, head_items = (n_units - tail_units) * nps;
    auto decode_item = [&](int item, int &unit, int &a, int &first, int &count) {
        int k;
        if (item < head_items) {
            unit = item / nps;
            k = item - unit * nps;
        } else {
            const int j = item - head_items;
            k = j / tail_units;
            unit = (n_units - tail_units) + (j - k * tail_units);
        }
        a = geo.ntq - 1 - 2 * k;
        first = geo.jmax(a);
        count = first + 1;
    };
    // number of key tiles of team 1 (0: no tile below)
    auto count1_of = [&](int a) { return a >= 1 ? geo.jmax(a - 1) + 1 : 0; };

    bool alive = true;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t it = 0, tg = 0, k_armed = 0, v_armed = 0, q_armed = 0;
            int item = (int)blockIdx.x;
            for (uint32_t k = 0; alive; ++k) {
                const uint32_t sl = k % kAttnSched, sph = (k / kAttnSched) & 1u;
                if (!mbar_wait(bar_sched_empty(sl), sph ^ 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                int unit = -1, a = 0, first = 0, count = 0;
                if (item < n_items) decode_item(item, unit, a, first, count);
                sched_s[sl] = make_int4(unit, a, first, count);
                mbar_arrive(bar_sched_full(sl));
                if (unit < 0) break;
                const int next = grid_n + atomicAdd(next_item, 1);
                for (int t = 0; t < count; ++t, ++tg) {
                    const uint32_t s = tg & 1u, ph = (tg >> 1) & 1u;
                    const int row0 = t * kTileRows;
                    if (!mbar_wait(bar_k_empty(s), ph ^ 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                    mbar_expect_tx(bar_k_full(s), kTile);
#pragma unroll
                    for (int bx = 0; bx < kBoxes; ++bx)
                        tma_load_3d(base + L::kK0 + s * kTile + bx * kBoxBytes, &map_k, bx * 64, row0, unit, bar_k_full(s));
                    k_armed = tg + 1;
                    if (t == 0) {
                        if (!mbar_wait(bar_q_empty, (it + 1u) & 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                        const int nq = a >= 1 ? 2 : 1;
                        mbar_expect_tx(bar_q_full, nq * kTile);
                        for (int x = 0; x < nq; ++x)
#pragma unroll
                            for (int bx = 0; bx < kBoxes; ++bx)
                                tma_load_3d(base + L::kQ0 + x * kTile + bx * kBoxBytes, &map_q, bx * 64, (a - x) * kTileRows, unit, bar_q_full);
                        q_armed = it + 1;
                    }
                    if (!mbar_wait(bar_v_empty(s), ph ^ 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                    mbar_expect_tx(bar_v_full(s), kTile);
#pragma unroll
                    for (int bx = 0; bx < kBoxes; ++bx)
                        tma_load_3d(base + L::kV0 + s * kTile + bx * kBoxBytes, &map_v, bx * 64, row0, unit, bar_v_full(s));
                    v_armed = tg + 1;
                }
                ++it;
                item = next;
            }
            if (*abort_flag) {
                // let copies that are still in flight land before the CTA gives its memory back
                if (q_armed > 0) mbar_wait(bar_q_full, (q_armed - 1u) & 1u, abort_flag, status, 200000ull);
                for (uint32_t t = k_armed > 2u ? k_armed - 2u : 0; t < k_armed; ++t)
                    mbar_wait(bar_k_full(t & 1u), (t >> 1) & 1u, abort_flag, status, 200000ull);
                for (uint32_t t = v_armed > 2u ? v_armed - 2u : 0; t < v_armed; ++t)
                    mbar_wait(bar_v_full(t & 1u), (t >> 1) & 1u, abort_flag, status, 200000ull);
            }
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t it = 0, tg = 0;
            uint32_t np[2] = {0, 0};            // per team: tiles whose P V was issued
            uint32_t ni[2] = {0, 0};            // per team: items it took part in
            // S of team x for the key tile in stage s (the caller has seen k_full of that stage)
            auto issue_s = [&](uint32_t x, uint32_t s) {
                const uint32_t a0 = base + L::kQ0 + x * kTile, b0 = base + L::kK0 + s * kTile;
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (uint32_t)(kk / 4) * kBoxBytes + (uint32_t)(kk % 4) * 32u;
                    umma_bf16(tmem_s(x), umma_desc(a0 + off), umma_desc(b0 + off), kIdescS, kk > 0 ? 1u : 0u);
                }
                umma_commit(bar_s_full(x));
            };
            for (uint32_t k = 0; alive; ++k) {
                const uint32_t sl = k % kAttnSched, sph = (k / kAttnSched) & 1u;
                if (!mbar_wait(bar_sched_full(sl), sph, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                const int4 d = sched_s[sl];
                mbar_arrive(bar_sched_empty(sl));
                if (d.x < 0) break;
                const int count = d.w, count1 = count1_of(d.y);
                if (!mbar_wait(bar_q_full, it & 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                // S of the first key tile for both teams
                if (!mbar_wait(bar_k_full(tg & 1u), (tg >> 1) & 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                tc_fence_after();
                issue_s(0, tg & 1u);
                if (count1 > 0) issue_s(1, tg & 1u);
                umma_commit(bar_k_empty(tg & 1u));
                if (count == 1) umma_commit(bar_q_empty);
                for (int t = 0; t < count; ++t, ++tg) {
                    const uint32_t s = tg & 1u, ph = (tg >> 1) & 1u;
                    const bool more = t + 1 < count;
                    const uint32_t s1 = (tg + 1u) & 1u, ph1 = ((tg + 1u) >> 1) & 1u;
                    for (uint32_t x = 0; x < 2; ++x) {
                        const int cnt_x = x == 0 ? count : count1;
                        if (t < cnt_x) {
                            // O += P V of team x for this key tile, then at once the team's S for the next one: both run
                            // while the other team does its softmax
                            if (!mbar_wait(bar_p_full(x), np[x] & 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                            if (!mbar_wait(bar_v_full(s), ph, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                            const bool first_of_item = t == 0;
                            // the team's previous output has been read out of TMEM before this item overwrites it
                            if (first_of_item && !mbar_wait(bar_o_free(x), (ni[x] + 1u) & 1u, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                            tc_fence_after();
                            const uint32_t v0 = base + L::kV0 + s * kTile;
#pragma unroll
                            for (int kk = 0; kk < kTileRows / 16; ++kk)      // 16 keys per instruction: 8 TMEM columns of P
                                umma_bf16_ts(tmem_o(x), tmem_s(x) + 8u * kk, umma_desc_mn(v0 + (uint32_t)kk * 2048u, kBoxBytes, 1024u),
                                             kIdescO, (!first_of_item || kk > 0) ? 1u : 0u);
                            ++np[x];
                            if (t + 1 == cnt_x) { umma_commit(bar_pv_done(x)); ++ni[x]; }    // the team's last product of the item
                        }
                        if (t + 1 < cnt_x) {
                            if (x == 0) {
                                if (!mbar_wait(bar_k_full(s1), ph1, abort_flag, status, kWaitLimitNs, kPollBackoffNs)) { alive = false; break; }
                                tc_fence_after();
                            }
                            issue_s(x, s1);
                        }
                    }
                    if (!alive) break;
                    umma_commit(bar_v_empty(s));                 // both teams' P V of this tile are issued
                    if (more) {
                        umma_commit(bar_k_empty(s1));            // and both teams' S of the next one
                        if (t + 2 == count) umma_commit(bar_q_empty);   // those were the item's last S: Q is free after them
                    }
                }
                ++it;
            }
        }
    } else {
        // ---------------------------------------------------------------- softmax warps
        const uint32_t x = (uint32_t)(warp - 2) >> 3;         // team
        const int q4 = warp & 3;                              // TMEM lane quarter this warp may access
        const int half = ((warp - 2) >> 2) & 1;               // which 64 columns of S, which half of O's columns
        const int r = q4 * 32 + lane;                         // row of the query tile = TMEM lane
        const uint32_t lane_sel = (uint32_t)(q4 * 32) << 16;
        const uint32_t s_addr = tmem_s(x) + lane_sel + (uint32_t)(half * 64);
        const uint32_t p_addr = tmem_s(x) + lane_sel + (uint32_t)(half * 32);    // 64 bf16 of P = 32 columns
        const uint32_t o_addr = tmem_o(x) + lane_sel + (uint32_t)(half * (D / 2));
        float *exch = exch_s + x * 2 * kTileRows;
        float *lsum = lsum_s + x * 2 * kTileRows;
        const float2 c2 = make_float2(c, c);
        uint32_t n = 0, ni = 0;                               // this team's tiles and items so far
        for (uint32_t k = 0; alive; ++k) {
            const uint32_t sl = k % kAttnSched, sph = (k / kAttnSched) & 1u;
            if (!mbar_wait(bar_sched_full(sl), sph, abort_flag, status)) { alive = false; break; }
            const int4 d = sched_s[sl];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_sched_empty(sl));
            if (d.x < 0) break;
            const int unit = d.x, st = d.y - (int)x;
            const int count = x == 0 ? d.w : count1_of(d.y);              // key tiles 0 .. count-1 for this team
            if (count == 0) continue;                                     // no tile for this team in this item
            float m_ref = -INFINITY, l = 0.f;                 // running maximum (log2 domain) and this half's row sum
            for (int t = 0; t < count; ++t, ++n) {
                const int off = (st - t) * kTileRows + geo.P;             // column col of key tile t is visible iff col <= r + off
                if (!mbar_wait(bar_s_full(x), n & 1u, abort_flag, status)) { alive = false; break; }
                tc_fence_after();
                float v[64];
                {
                    uint32_t ra[32], rb[32];
                    tmem_ld32_async(s_addr, ra);
                    tmem_ld32_async(s_addr + 32, rb);
                    tmem_ld_wait(ra);
                    tmem_ld_wait(rb);
#pragma unroll
                    for (int i = 0; i < 32; ++i) { v[i] = __uint_as_float(ra[i]); v[32 + i] = __uint_as_float(rb[i]); }
                }
                if (off < kTileRows - 1) {
                    const int lim = r + off - half * 64;
#pragma unroll
                    for (int i = 0; i < 64; ++i) if (i > lim) v[i] = -INFINITY;
                }
                float mx4[4] = {v[0], v[1], v[2], v[3]};
#pragma unroll
                for (int i = 4; i < 64; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], v[i]);
                const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                // Both halves of the row agree on the tile's maximum before either scales anything. Passing
                // this rendezvous also means that every thread of the team holds its part of S in registers:
                // from here on P may be written over S.
                exch[half * kTileRows + r] = mx;
                mbar_arrive(bar_x_rdv(x));
                if (!mbar_wait(bar_x_rdv(x), n & 1u, abort_flag, status)) { alive = false; break; }
                const float tile_max = fmaxf(mx, exch[(half ^ 1) * kTileRows + r]) * c;
                float factor = 1.f;
                bool rescale = false;
                if (tile_max > m_ref + kRaiseBy) {            // also the first tile that shows this row anything
                    if (m_ref != -INFINITY) { rescale = true; factor = fast_exp2(m_ref - tile_max); }
                    m_ref = tile_max;
                }
                const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                const float2 nm = make_float2(-m_use, -m_use);
                float2 sum2 = make_float2(0.f, 0.f);
                uint32_t pk[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float2 a = __ffma2_rn(make_float2(v[2 * i], v[2 * i + 1]), c2, nm);
                    const float2 e = exp2_pair(a, i);
                    sum2 = __fadd2_rn(sum2, e);
                    pk[i] = pack2(e.x, e.y);
                }
                l = l * factor + (sum2.x + sum2.y);
                // This tile's S was issued behind the previous tile's P V, and the tensor cores complete in
                // issue order: O is at rest and the previous P has been consumed.
                // TMEM loads and stores are warp-wide instructions: if any row of the warp raises its maximum,
                // the whole warp rescales (the other rows multiply by one, which changes nothing).
                if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
                    for (int j = 0; j < D / 64; ++j) {
                        uint32_t ro[32];
                        tmem_ld32_async(o_addr + 32 * j, ro);
                        tmem_ld_wait(ro);
#pragma unroll
                        for (int i = 0; i < 32; ++i) ro[i] = __float_as_uint(__uint_as_float(ro[i]) * factor);
                        tmem_st32(o_addr + 32 * j, ro);
                    }
                }
                tmem_st32(p_addr, pk);
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_p_full(x));
            }
            if (!alive) break;

            // the item's last P V has completed: normalise and store the rows, report the normaliser
            if (!mbar_wait(bar_pv_done(x), ni & 1u, abort_flag, status)) { alive = false; break; }
            tc_fence_after();
            lsum[half * kTileRows + r] = l;
            mbar_arrive(bar_l_rdv(x));
            if (!mbar_wait(bar_l_rdv(x), ni & 1u, abort_flag, status)) { alive = false; break; }
            const float l_tot = l + lsum[(half ^ 1) * kTileRows + r];
            const float inv = l_tot > 0.f ? 1.f / l_tot : 0.f;
            const int row = st * kTileRows + r;
#pragma unroll
            for (int j = 0; j < D / 64; ++j) {
                uint32_t ro[32];
                tmem_ld32_async(o_addr + 32 * j, ro);
                tmem_ld_wait(ro);
                if (row < geo.Tq) {
                    __nv_bfloat16 *dst = out + ((size_t)unit * geo.Tq + row) * D + half * (D / 2) + 32 * j;
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        float f[8], g[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            f[i] = __uint_as_float(ro[16 * q + i]) * inv;
                            g[i] = __uint_as_float(ro[16 * q + 8 + i]) * inv;
                        }
                        st_global_32B(dst + 16 * q, pack8(f), pack8(g));
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_o_free(x));
            if (half == 0) {
                const float l2 = (row < geo.Tq) ? m_ref + __log2f(l_tot) : INFINITY;
                lse2[(size_t)unit * geo.ntq * kTileRows + row] = l2;                 // padded layout of the column-sum pass
                if (lse_out && row < geo.Tq) lse_out[(size_t)unit * geo.Tq + row] = l2 * kLn2;
            }
            ++ni;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)kAttnTmemCols) : "memory");
    }
}

template <int D>
cudaError_t launch_attention_t(const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mv, int units,
                               const Geometry &geo, float c, void *out, float *lse2, float *lse_out, int *status,
                               cudaStream_t stream)
{
    constexpr int smem = AttnSmem<D>::kDynBytes;
    cudaError_t e = cudaFuncSetAttribute(attention_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    const long long resident = sm_count();                        // one persistent CTA per SM
    const int nps = (geo.ntq + 1) / 2;                            // items (pairs of query tiles) per unit
    const long long items = (long long)units * nps;
    const unsigned grid = (unsigned)(items < resident ? items : resident);
    const long long tail = (3 * resident + nps - 1) / nps;
    attention_kernel<D><<<grid, kAttnThreads, smem, stream>>>(mq, mk, mv, geo, (int)items, (int)(tail < units ? tail : units), c,
                                                              static_cast<__nv_bfloat16 *>(out), lse2, lse_out, status,
                                                              status + 3);
    return cudaGetLastError();
}

}  // namespace

// Q: [units, Tq, D]; K, V: [units, P + Tq, D]; out: [units, Tq, D] bf16; lse_out (nullable): [units, Tq].
// Leaves the padded log2-domain normaliser in the workspace (behind the status block), where the
// column-sum pass of the importance kernels reads it. Zeroes the status block first.
cudaError_t launch_attention(const void *Q, const void *K, const void *V, void *out, float *lse_out, int N, int H,
                             int Tq, int P, int D, float scale, void *ws, cudaStream_t stream)
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
    if ((long long)units * geo.ntk > 0x7FFF0000LL) return cudaErrorInvalidConfiguration;
    CUtensorMap mq, mk, mv;
    if (!make_map(&mq, Q, units, Tq, D) || !make_map(&mk, K, units, Tq + P, D) || !make_map(&mv, V, units, Tq + P, D))
        return cudaErrorInvalidValue;
    const float c = scale * kLog2e;
    if (D == 128) return launch_attention_t<128>(mq, mk, mv, units, geo, c, out, lse2, lse_out, status, stream);
    return launch_attention_t<64>(mq, mk, mv, units, geo, c, out, lse2, lse_out, status, stream);
}

}  // namespace ec
