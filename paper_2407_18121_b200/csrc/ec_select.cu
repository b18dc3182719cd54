// Anchor selection (Sec. 3.3: the N_I positions with the highest importance, ascending)
// as an exact radix select on fp32 bit patterns followed by an order-preserving compaction.
#include "ec_common.cuh"

namespace ec {

namespace {

constexpr int kSelThreads = 256;

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
    const size_t grp = blockIdx.y;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const float *s = scores + grp * share * T + t;
    float acc = 0.f;
    for (int j = 0; j < share; ++j) acc += s[(size_t)j * T];
    mean[grp * T + t] = acc / (float)share;
}

// One CTA per selection unit. Dynamic shared memory: T keys + n_keep anchors.
// `replicate` > 1 writes the same anchors for that many consecutive heads (layer-shared mode).
__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float *__restrict__ scores, int T, int C, int protect_ends, int replicate,
              int32_t *__restrict__ anchor_pos, int32_t *__restrict__ bucket_len)
{
    extern __shared__ uint32_t smem[];
    uint32_t *keys = smem;
    int32_t *anch = reinterpret_cast<int32_t *>(smem + T);
    __shared__ uint32_t hist[256];
    __shared__ uint32_t s_prefix, s_need;
    __shared__ uint32_t warp_gt[kSelThreads / 32], warp_eq[kSelThreads / 32];

    const int tid = threadIdx.x;
    const size_t unit = blockIdx.x;
    const float *s = scores + unit * T;

    // Protected positions (first and last) are always anchors: they get the top key and are left
    // out of the search for the threshold among the others.
    auto is_prot = [&](int t) { return protect_ends && (t == 0 || (t == T - 1 && C >= 2)); };
    const int nprot = protect_ends ? ((C >= 2 && T >= 2) ? 2 : 1) : 0;
    const uint32_t need0 = (uint32_t)(C - nprot);        // anchors still to find among unprotected keys

    uint32_t kmin = 0xFFFFFFFFu, kmax = 0u;
    for (int t = tid; t < T; t += kSelThreads) {
        uint32_t k = sort_key(s[t]);
        if (is_prot(t)) k = 0xFFFFFFFFu;
        else { kmin = min(kmin, k); kmax = max(kmax, k); }
        keys[t] = k;
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        kmin = min(kmin, __shfl_xor_sync(0xFFFFFFFFu, kmin, o));
        kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, o));
    }
    if ((tid & 31) == 0) { warp_gt[tid >> 5] = kmin; warp_eq[tid >> 5] = kmax; }   // reused below for the scan
    __syncthreads();
    kmin = warp_gt[0];
    kmax = warp_eq[0];
#pragma unroll
    for (int w = 1; w < kSelThreads / 32; ++w) { kmin = min(kmin, warp_gt[w]); kmax = max(kmax, warp_eq[w]); }
    __syncthreads();

    // Radix select for the need0-th largest unprotected key. All keys agree on the bits above the
    // highest bit in which the smallest and the largest key differ, so only the bits below it are
    // examined, 8 at a time from the top: the digits spread over the keys' real range (attention
    // column sums lie within a few octaves, so a fixed top byte would put them all in a few bins).
    if (need0 == 0) {
        if (tid == 0) { s_prefix = 0xFFFFFFFEu; s_need = 0; }             // only the protected keys pass
    } else if (kmin == kmax) {
        if (tid == 0) { s_prefix = kmin; s_need = need0; }                // every key is a tie
    } else {
        const int nbits = 32 - __clz(kmin ^ kmax);                        // bits that vary: [nbits-1 .. 0]
        const int passes = (nbits + 7) / 8;
        if (tid == 0) {
            s_prefix = (nbits == 32) ? 0u : (kmax >> nbits) << nbits;     // the common high bits
            s_need = need0;
        }
        for (int pass = 0; pass < passes; ++pass) {
            const int shift = 8 * (passes - 1 - pass);
            const int width = (pass == 0) ? nbits - shift : 8;            // the top digit may be narrower
            const uint32_t dmask = (1u << width) - 1u;
            const uint32_t himask = (shift + width >= 32) ? 0u : (0xFFFFFFFFu << (shift + width));
            hist[tid] = 0;                       // kSelThreads == 256 bins
            __syncthreads();
            const uint32_t prefix = s_prefix, need = s_need;
            for (int t = tid; t < T; t += kSelThreads) {
                const uint32_t k = keys[t];
                if ((k & himask) == (prefix & himask) && !is_prot(t)) atomicAdd(&hist[(k >> shift) & dmask], 1u);
            }
            __syncthreads();
            if (tid < 32) {
                // lane l owns bins 255-8l .. 248-8l (descending); suffix-scan across lanes
                uint32_t local[8], sum = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) { local[i] = hist[255 - (tid * 8 + i)]; sum += local[i]; }
                uint32_t incl = sum;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                    if (tid >= o) incl += v;
                }
                uint32_t before = incl - sum;    // keys in strictly higher bins than this lane's
                if (before < need && need <= incl) {
                    uint32_t run = before;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        if (run < need && need <= run + local[i]) {
                            s_prefix = prefix | ((uint32_t)(255 - (tid * 8 + i)) << shift);
                            s_need = need - run;  // how many are still needed inside this bin
                        }
                        run += local[i];
                    }
                }
            }
            __syncthreads();
        }
    }
    __syncthreads();
    const uint32_t thr = s_prefix;       // key of the last anchor taken by score (protected keys lie above it)
    const uint32_t need_eq = s_need;     // how many keys equal to thr are taken (lowest positions)

    // Ordered compaction: thread i owns the contiguous positions [i*ipt, (i+1)*ipt).
    const int ipt = (T + kSelThreads - 1) / kSelThreads;
    const int t0 = min(tid * ipt, T), t1 = min(t0 + ipt, T);
    uint32_t gt = 0, eq = 0;
    for (int t = t0; t < t1; ++t) {
        uint32_t k = keys[t];
        gt += (k > thr);
        eq += (k == thr);
    }
    uint32_t gt_incl = gt, eq_incl = eq;
    const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t a = __shfl_up_sync(0xFFFFFFFFu, gt_incl, o);
        uint32_t b = __shfl_up_sync(0xFFFFFFFFu, eq_incl, o);
        if (lane >= o) { gt_incl += a; eq_incl += b; }
    }
    if (lane == 31) { warp_gt[warp] = gt_incl; warp_eq[warp] = eq_incl; }
    __syncthreads();
    uint32_t gt_before = gt_incl - gt, eq_before = eq_incl - eq;
    for (int w = 0; w < warp; ++w) { gt_before += warp_gt[w]; eq_before += warp_eq[w]; }
    for (int t = t0; t < t1; ++t) {
        uint32_t k = keys[t];
        if (k > thr) {
            anch[gt_before + min(eq_before, need_eq)] = t;
            ++gt_before;
        } else if (k == thr) {
            if (eq_before < need_eq) anch[gt_before + eq_before] = t;
            ++eq_before;
        }
    }
    __syncthreads();

    // the merge kernel behind this one may start scheduling; it waits for this grid to finish
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int r = 0; r < replicate; ++r) {
        int32_t *ap = anchor_pos + (unit * replicate + r) * C;
        for (int k = tid; k < C; k += kSelThreads) ap[k] = anch[k];
        if (bucket_len) {
            // Eq. 2: bucket k spans floor((t_{k-1}+t_k)/2)+1 .. floor((t_k+t_{k+1})/2)
            int32_t *bl = bucket_len + (unit * replicate + r) * C;
            for (int k = tid; k < C; k += kSelThreads) {
                int lo = (k == 0) ? 0 : ((anch[k - 1] + anch[k]) >> 1) + 1;
                int hi = (k == C - 1) ? T - 1 : ((anch[k] + anch[k + 1]) >> 1);
                bl[k] = hi - lo + 1;
            }
        }
    }
}

}  // namespace

// `share` consecutive units rank one common (averaged) score vector; share == 1: every unit its own.
cudaError_t launch_select(const float *scores, int units, int T, int n_keep, int share, int protect_ends,
                          int32_t *anchor_pos, int32_t *bucket_len, float *mean_ws, cudaStream_t stream)
{
    size_t smem = (size_t)(T + n_keep) * sizeof(uint32_t);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    if (share > 1) {
        const int groups = units / share;
        if (groups > 65535) return cudaErrorInvalidConfiguration;
        dim3 g((T + 255) / 256, groups);
        group_mean_kernel<<<g, 256, 0, stream>>>(scores, mean_ws, share, T);
        select_kernel<<<groups, kSelThreads, smem, stream>>>(mean_ws, T, n_keep, protect_ends, share, anchor_pos, bucket_len);
    } else {
        select_kernel<<<units, kSelThreads, smem, stream>>>(scores, T, n_keep, protect_ends, 1, anchor_pos, bucket_len);
    }
    return cudaGetLastError();
}

}  // namespace ec
