// Bucket division (Eq. 2) and mean merge (Eq. 3) into the dense compacted cache.
// HBM-bound streaming: every prompt row of K and V is read exactly once with 16-byte loads,
// every kept row is written once.
#include "ec_common.cuh"

namespace ec {

namespace {

constexpr int kMergeThreads = 256;
constexpr int kRowsPerCta = 64;   // output rows (buckets) handled by one CTA

// LPR = lanes per row = D / 8 (each lane holds 8 bf16 = 16 bytes of a row).
// grid.x = units * chunks; a lane group walks buckets k0+g, k0+g+G, ... of its chunk and
// sums the bucket's rows in position order in fp32.
template <int LPR>
__global__ void __launch_bounds__(kMergeThreads)
merge_kernel(const uint4 *__restrict__ K, const uint4 *__restrict__ V, const int32_t *__restrict__ anchor_pos,
             int T, int C, int chunks, uint4 *__restrict__ Kc, uint4 *__restrict__ Vc, int cap)
{
    constexpr int G = kMergeThreads / LPR;          // lane groups per CTA
    const int unit = blockIdx.x / chunks;
    const int chunk = blockIdx.x - unit * chunks;
    const int g = threadIdx.x / LPR;
    const int l = threadIdx.x - g * LPR;
    const int32_t *anch = anchor_pos + (size_t)unit * C;
    const uint4 *Ku = K + (size_t)unit * T * LPR;
    const uint4 *Vu = V + (size_t)unit * T * LPR;
    uint4 *Kcu = Kc + (size_t)unit * cap * LPR;
    uint4 *Vcu = Vc + (size_t)unit * cap * LPR;

    const int k_end = min((chunk + 1) * kRowsPerCta, C);
    for (int k = chunk * kRowsPerCta + g; k < k_end; k += G) {
        const int a = anch[k];
        const int lo = (k == 0) ? 0 : ((anch[k - 1] + a) >> 1) + 1;
        const int hi = (k == C - 1) ? T - 1 : ((a + anch[k + 1]) >> 1);
        float ak[8], av[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) { ak[i] = 0.f; av[i] = 0.f; }
        int t = lo;
        for (; t + 3 <= hi; t += 4) {
            uint4 rk[4], rv[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                rk[j] = ldg_stream(Ku + (size_t)(t + j) * LPR + l);
                rv[j] = ldg_stream(Vu + (size_t)(t + j) * LPR + l);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                float fk[8], fv[8];
                unpack8(rk[j], fk);
                unpack8(rv[j], fv);
#pragma unroll
                for (int i = 0; i < 8; ++i) { ak[i] += fk[i]; av[i] += fv[i]; }
            }
        }
        for (; t <= hi; ++t) {
            uint4 rk = ldg_stream(Ku + (size_t)t * LPR + l);
            uint4 rv = ldg_stream(Vu + (size_t)t * LPR + l);
            float fk[8], fv[8];
            unpack8(rk, fk);
            unpack8(rv, fv);
#pragma unroll
            for (int i = 0; i < 8; ++i) { ak[i] += fk[i]; av[i] += fv[i]; }
        }
        const float cnt = (float)(hi - lo + 1);
#pragma unroll
        for (int i = 0; i < 8; ++i) { ak[i] = ak[i] / cnt; av[i] = av[i] / cnt; }
        Kcu[(size_t)k * LPR + l] = pack8(ak);
        Vcu[(size_t)k * LPR + l] = pack8(av);
    }
}

}  // namespace

cudaError_t launch_merge(const void *K, const void *V, const int32_t *anchor_pos, int units, int T, int D,
                         int n_keep, void *Kc, void *Vc, int cap, cudaStream_t stream)
{
    const int chunks = (n_keep + kRowsPerCta - 1) / kRowsPerCta;
    const long long grid = (long long)units * chunks;
    if (grid > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    if (D == 128) {
        merge_kernel<16><<<(unsigned)grid, kMergeThreads, 0, stream>>>(
            (const uint4 *)K, (const uint4 *)V, anchor_pos, T, n_keep, chunks, (uint4 *)Kc, (uint4 *)Vc, cap);
    } else {
        merge_kernel<8><<<(unsigned)grid, kMergeThreads, 0, stream>>>(
            (const uint4 *)K, (const uint4 *)V, anchor_pos, T, n_keep, chunks, (uint4 *)Kc, (uint4 *)Vc, cap);
    }
    return cudaGetLastError();
}

}  // namespace ec
