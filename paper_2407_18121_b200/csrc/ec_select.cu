// Anchor selection (Sec. 3.3: the N_I positions with the highest importance, ascending):
// a warp-level radix select over bit planes held in registers finds the exact N_I-th largest fp32
// bit pattern, then warp ballots list the anchors in position order.
#include "ec_common.cuh"

namespace ec {

namespace {

// Order-preserving map from fp32 to uint32 (larger float -> larger key).
__device__ __forceinline__ uint32_t sort_key(float x)
{
    uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Shared population: mean over `share` consecutive units (the heads of a layer, or every
// layer and head of a sequence). scores [G*share, T] -> mean [G, T].
__global__ void group_mean_kernel(const float *__restrict__ scores, float *__restrict__ mean, int share, int T)
{
    const size_t grp = blockIdx.x;
    const int t = blockIdx.y * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const float *s = scores + grp * share * T + t;
    float acc = 0.f;
    for (int j = 0; j < share; ++j) acc += s[(size_t)j * T];
    mean[grp * T + t] = acc / (float)share;
}

constexpr int kKeysPerLane = 32;                        // a warp holds 1024 consecutive positions
constexpr int kWarpSpan = 32 * kKeysPerLane;
constexpr int kMaxWarpsPerUnit = 16;                    // T <= 16384

// Transpose of a 32 x 32 bit matrix held as one column of shared memory per lane (word i of the
// lane = m[i * 32], row i of the matrix; column c = bit 31 - c): five butterfly stages of masked
// swaps between words. Kept as loops on purpose: a selection warp runs this code once, so compact
// code (few instruction-cache misses) matters more than instruction count.
__device__ __forceinline__ void transpose32(uint32_t *m)
{
    uint32_t mask = 0x0000FFFFu;
#pragma unroll 1
    for (int j = 16; j != 0; j >>= 1) {
#pragma unroll 1
        for (int h = 0; h < 16; h += 8) {              // eight word pairs at a time: all loads, then all stores,
            uint32_t lo[8], hi[8];                      // so that the loads do not queue behind the stores
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int k = (((h + i) & ~(j - 1)) << 1) | ((h + i) & (j - 1));   // (h+i)-th index with bit j clear
                lo[i] = m[k * 32];
                hi[i] = m[(k + j) * 32];
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int k = (((h + i) & ~(j - 1)) << 1) | ((h + i) & (j - 1));
                const uint32_t t = (lo[i] ^ (hi[i] >> j)) & mask;
                m[k * 32] = lo[i] ^ t;
                m[(k + j) * 32] = hi[i] ^ (t << j);
            }
        }
        mask ^= mask << (j >> 1);
    }
}

// Warp-level selection. G warps share one unit (G = ceil(T / 1024)); with G == 1 a CTA holds four
// independent units, one per warp, and no block-wide barrier is ever needed. Lane l of warp w owns
// positions 1024*w + 32*j + l (j = 0..31, its "rows").
//  1. The lane's 32 keys (order-preserving uint32 images of the scores) are transposed into 32
//     bit planes (a shared-memory column per lane), so "how many of my still-undecided keys have bit b set" is one AND and one popc.
//  2. Radix descent from the top bit for the C-th largest key: if at least `need` undecided keys of
//     the unit have the bit set, those stay undecided and the others are out; otherwise they are all
//     anchors (`greater`), `need` shrinks by their count and the others stay undecided. All keys
//     agree on the bits above the highest bit in which the smallest and the largest key differ, so
//     the descent starts there and takes two bits per step (the three counts of a step need one
//     round of warp reductions). What is still undecided at the end equals the threshold: ties, of
//     which the `need` lowest positions are taken. Protected positions (first, last) are anchors
//     from the start.
//  3. Ordered compaction with warp ballots, one row of 32 consecutive positions at a time.
// `replicate` > 1 writes the same anchors for that many consecutive heads (shared populations).
template <int G>
__global__ void __launch_bounds__(G == 1 ? 128 : 32 * G)
select_kernel(const float *__restrict__ scores, int n_units, int T, int C, int protect_ends, int replicate,
              int32_t *__restrict__ anchor_pos, int32_t *__restrict__ bucket_len)
{
    __shared__ uint32_t xa[2][kMaxWarpsPerUnit], xc[2][kMaxWarpsPerUnit];   // cross-warp exchange (G > 1), double-buffered
    extern __shared__ uint32_t planes_all[];                               // 32 x 32 words per warp
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // launched with programmatic stream serialization: the kernel in front (normally the importance
    // kernel's column-sum pass) must have finished before the scores are read
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int unit = (G == 1) ? blockIdx.x * 4 + warp : blockIdx.x;
    if (G == 1 && unit >= n_units) return;                 // whole warp leaves; no barriers in this variant
    const int wu = (G == 1) ? 0 : warp;                    // this warp's index inside the unit
    const int base = wu * kWarpSpan;
    const float *s = scores + (size_t)unit * T;

    auto is_prot = [&](int t) { return protect_ends && (t == 0 || (t == T - 1 && C >= 2)); };
    const int nprot = protect_ends ? ((C >= 2 && T >= 2) ? 2 : 1) : 0;
    int par = 0;
    auto unit_sum = [&](uint32_t v) {                      // sum over the unit's warps, same value in every thread
        v = __reduce_add_sync(0xFFFFFFFFu, v);
        if (G == 1) return v;
        if (lane == 0) xa[par][wu] = v;
        __syncthreads();                                   // buffers alternate: one barrier per use
        uint32_t t = 0;
#pragma unroll
        for (int w = 0; w < G; ++w) t += xa[par][w];
        par ^= 1;
        return t;
    };
    auto unit_sum2 = [&](uint32_t &a, uint32_t &b) {       // two sums for the price of one barrier
        a = __reduce_add_sync(0xFFFFFFFFu, a);
        b = __reduce_add_sync(0xFFFFFFFFu, b);
        if (G == 1) return;
        if (lane == 0) { xa[par][wu] = a; xc[par][wu] = b; }
        __syncthreads();
        a = 0; b = 0;
#pragma unroll
        for (int w = 0; w < G; ++w) { a += xa[par][w]; b += xc[par][w]; }
        par ^= 1;
    };

    // pl[(31 - j) * 32] = key of row j, so that after the transpose pl[(31 - b) * 32] is the plane of
    // key bit b with row j at mask bit j (one shared-memory column per lane: conflict-free)
    uint32_t *pl = planes_all + warp * 1024 + lane;
    uint32_t undecided = 0u, greater = 0u;                 // row masks
    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;               // range of the unprotected keys
    {
        float raw[kKeysPerLane];
#pragma unroll
        for (int j = 0; j < kKeysPerLane; ++j) {           // all loads first, so that they overlap
            const int t = base + 32 * j + lane;
            raw[j] = (t < T) ? __ldg(s + t) : 0.f;
        }
#pragma unroll
        for (int j = 0; j < kKeysPerLane; ++j) {
            const int t = base + 32 * j + lane;
            uint32_t key = 0u;
            if (t < T) {
                key = sort_key(raw[j]);
                if (is_prot(t)) greater |= 1u << j;
                else { undecided |= 1u << j; kmin = min(kmin, key); kmax = max(kmax, key); }
            }
            pl[(31 - j) * 32] = key;
        }
    }
    kmin = __reduce_min_sync(0xFFFFFFFFu, kmin);
    kmax = __reduce_max_sync(0xFFFFFFFFu, kmax);
    if (G > 1) {
        if (lane == 0) { xa[par][wu] = kmin; xc[par][wu] = kmax; }
        __syncthreads();
#pragma unroll
        for (int w = 0; w < G; ++w) { kmin = min(kmin, xa[par][w]); kmax = max(kmax, xc[par][w]); }
        par ^= 1;
    }
    transpose32(pl);

    uint32_t need = (uint32_t)(C - nprot);                // anchors still to find among the unprotected keys
    if (need == 0) {
        undecided = 0u;                                   // only the protected keys are anchors
    } else if (kmin != kmax) {                            // (kmin == kmax: every unprotected key is a tie)
        const int nbits = 32 - __clz(kmin ^ kmax);
        int b = nbits - 1;
#pragma unroll 1
        for (; b >= 1; b -= 2) {                          // two bits per step; uniform over the unit
            const uint32_t p1 = pl[(31 - b) * 32], p0 = pl[(32 - b) * 32];
            const uint32_t u11 = undecided & p1 & p0, u10 = undecided & p1 & ~p0, u01 = undecided & ~p1 & p0;
            // counts of the three non-zero patterns: c11 and c10 share a word (a unit has at most
            // 16384 keys, so the 16-bit fields cannot carry into each other)
            uint32_t packed = (uint32_t)__popc(u11) | ((uint32_t)__popc(u10) << 16), c01 = (uint32_t)__popc(u01);
            unit_sum2(packed, c01);
            const uint32_t c11 = packed & 0xFFFFu, c10 = packed >> 16;
            if (c11 >= need) {
                undecided = u11;
            } else if (c11 + c10 >= need) {
                need -= c11; greater |= u11; undecided = u10;
            } else if (c11 + c10 + c01 >= need) {
                need -= c11 + c10; greater |= u11 | u10; undecided = u01;
            } else {
                need -= c11 + c10 + c01; greater |= u11 | u10 | u01; undecided &= ~(p1 | p0);
            }
        }
        if (b == 0) {                                     // an odd number of bits: the last one alone
            const uint32_t plane = pl[31 * 32];
            const uint32_t ones = undecided & plane;
            const uint32_t c1 = unit_sum(__popc(ones));
            if (c1 >= need) {
                undecided = ones;
            } else {
                need -= c1;
                greater |= ones;
                undecided &= ~plane;
            }
        }
    }
    const uint32_t need_eq = need;                        // ties taken, lowest positions first

    // anchors / ties held by earlier warps of the unit
    uint32_t gb = 0, eb = 0;
    if (G > 1) {
        const uint32_t gt = __reduce_add_sync(0xFFFFFFFFu, __popc(greater));
        const uint32_t eq = __reduce_add_sync(0xFFFFFFFFu, __popc(undecided));
        if (lane == 0) { xa[par][wu] = gt; xc[par][wu] = eq; }
        __syncthreads();
#pragma unroll
        for (int w = 0; w < G; ++w)
            if (w < wu) { gb += xa[par][w]; eb += xc[par][w]; }
        par ^= 1;
    }

    const uint32_t lt_mask = (1u << lane) - 1u;
    int32_t *ap0 = anchor_pos + (size_t)unit * replicate * C;
    const int rows = min(kKeysPerLane, (T - base + 31) >> 5);          // rows of this warp that hold positions < T
#pragma unroll 4
    for (int j = 0; j < rows; ++j) {
        const bool is_gt = (greater >> j) & 1u, is_eq = (undecided >> j) & 1u;
        const uint32_t bg = __ballot_sync(0xFFFFFFFFu, is_gt), be = __ballot_sync(0xFFFFFFFFu, is_eq);
        const uint32_t g_here = gb + __popc(bg & lt_mask), e_here = eb + __popc(be & lt_mask);
        // anchors before this position = its own index; one predicated store, no divergent code
        const bool take = is_gt || (is_eq && e_here < need_eq);
        const int idx = (int)(g_here + min(e_here, need_eq));
        if (take) ap0[idx] = base + 32 * j + lane;
        gb += __popc(bg);
        eb += __popc(be);
    }

    // the merge kernel behind this one may start scheduling; it waits for this grid to finish
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (bucket_len || replicate > 1) {
        // the anchors just written by the unit's own warps are visible after the barrier
        if (G == 1) __syncwarp(); else __syncthreads();
        const volatile int32_t *av = ap0;
        for (int kk = wu * 32 + lane; kk < C; kk += 32 * G) {
            const int c0 = av[kk];
            for (int r = 1; r < replicate; ++r) ap0[(size_t)r * C + kk] = c0;       // shared population: same anchors
            if (bucket_len) {
                // Eq. 2: bucket k spans floor((t_{k-1}+t_k)/2)+1 .. floor((t_k+t_{k+1})/2)
                const int lo = (kk == 0) ? 0 : ((av[kk - 1] + c0) >> 1) + 1;
                const int hi = (kk == C - 1) ? T - 1 : ((c0 + av[kk + 1]) >> 1);
                for (int r = 0; r < replicate; ++r) bucket_len[((size_t)unit * replicate + r) * C + kk] = hi - lo + 1;
            }
        }
    }
}

}  // namespace

namespace {
template <int G>
cudaError_t launch_select_t(const float *scores, int n_units, int T, int n_keep, int protect_ends, int replicate,
                            int32_t *anchor_pos, int32_t *bucket_len, cudaStream_t stream)
{
    const unsigned grid = (G == 1) ? (unsigned)((n_units + 3) / 4) : (unsigned)n_units;
    constexpr int smem = (G == 1 ? 4 : G) * 32 * 32 * (int)sizeof(uint32_t);      // bit planes: 4 KB per warp
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(select_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(G == 1 ? 128 : 32 * G);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, select_kernel<G>, scores, n_units, T, n_keep, protect_ends, replicate, anchor_pos, bucket_len);
}
}  // namespace

// `share` consecutive units rank one common (averaged) score vector; share == 1: every unit its own.
cudaError_t launch_select(const float *scores, int units, int T, int n_keep, int share, int protect_ends,
                          int32_t *anchor_pos, int32_t *bucket_len, float *mean_ws, cudaStream_t stream)
{
    const float *src = scores;
    int n = units, rep = 1;
    if (share > 1) {
        const int groups = units / share;
        dim3 g(groups, (T + 255) / 256);
        group_mean_kernel<<<g, 256, 0, stream>>>(scores, mean_ws, share, T);
        src = mean_ws;
        n = groups;
        rep = share;
    }
    const int G = (T + kWarpSpan - 1) / kWarpSpan;
    switch (G) {
    case 1: return launch_select_t<1>(src, n, T, n_keep, protect_ends, rep, anchor_pos, bucket_len, stream);
    case 2: return launch_select_t<2>(src, n, T, n_keep, protect_ends, rep, anchor_pos, bucket_len, stream);
    case 3: case 4: return launch_select_t<4>(src, n, T, n_keep, protect_ends, rep, anchor_pos, bucket_len, stream);
    case 5: case 6: case 7: case 8: return launch_select_t<8>(src, n, T, n_keep, protect_ends, rep, anchor_pos, bucket_len, stream);
    default: break;
    }
    if (G > kMaxWarpsPerUnit) return cudaErrorInvalidConfiguration;
    return launch_select_t<16>(src, n, T, n_keep, protect_ends, rep, anchor_pos, bucket_len, stream);
}

}  // namespace ec
