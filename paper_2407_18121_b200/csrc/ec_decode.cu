// Decode attention over the compacted cache plus the step's new row, with the new row
// written into the slot freed by fixed-point elimination (Sec. 3.3 "Output Generation").
// HBM-bound: every cached K and V row is read once per step with 16-byte loads.
#include "ec_common.cuh"

namespace ec {

namespace {

// Tunables (compile-time): threads per CTA and cache rows a lane group fetches per iteration.
// 128-thread CTAs keep at least 7 CTAs resident per SM, so that the 1024 units of a 7B-shaped
// single-sequence step (6.9 per SM) all run in one balanced wave.
#ifndef EC_DEC_THREADS
#define EC_DEC_THREADS 128
#endif
#ifndef EC_DEC_ROWS
#define EC_DEC_ROWS 4
#endif
#ifndef EC_DEC_MIN_CTAS
#define EC_DEC_MIN_CTAS 7
#endif
constexpr int kDecThreads = EC_DEC_THREADS;
constexpr int kRowsPerIter = EC_DEC_ROWS;

// The cache is written later in the same kernel, so no read-only (.nc) path here.
__device__ __forceinline__ uint4 ld_row(const uint4 *p)
{
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// grid.x = units * splits. Rows 0..len-1 come from the cache, row `len` is the new token.
// LPR lanes share one row (8 bf16 each); a lane group keeps a running (max, sum, acc) in
// the log2 domain and the CTA merges its groups through shared memory.
// splits == 1: writes out (bf16) and stores the new row into `write_slot`.
// splits  > 1: writes (acc[D], max, sum) per split to `partials`; the combine kernel finishes.
template <int LPR>
__global__ void __launch_bounds__(kDecThreads, EC_DEC_MIN_CTAS)
decode_kernel(const uint4 *__restrict__ q, const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new,
              uint4 *Kc, uint4 *Vc, int cap, int len, int write_slot, float scale_log2e,
              __nv_bfloat16 *__restrict__ out, float *__restrict__ partials, int splits)
{
    constexpr int D = LPR * 8;
    constexpr int G = kDecThreads / LPR;
    __shared__ float sm_acc[G][D];
    __shared__ float sm_m[G], sm_l[G];

    const int unit = blockIdx.x / splits;
    const int split = blockIdx.x - unit * splits;
    const int g = threadIdx.x / LPR;
    const int l = threadIdx.x - g * LPR;
    const unsigned gmask = ((LPR == 16) ? 0xFFFFu : 0xFFu) << ((threadIdx.x & 31) / LPR * LPR);

    uint4 *Kcu = Kc + (size_t)unit * cap * LPR;
    uint4 *Vcu = Vc + (size_t)unit * cap * LPR;
    const uint4 *knu = k_new + (size_t)unit * LPR;
    const uint4 *vnu = v_new + (size_t)unit * LPR;

    float qf[8];
    unpack8(q[(size_t)unit * LPR + l], qf);
#pragma unroll
    for (int i = 0; i < 8; ++i) qf[i] *= scale_log2e;

    const int rows = len + 1;
    const int per = (rows + splits - 1) / splits;
    const int r0 = split * per, r1 = min(r0 + per, rows);

    float m = -INFINITY, lsum = 0.f, acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;

    for (int j0 = r0 + g * kRowsPerIter; j0 < r1; j0 += G * kRowsPerIter) {
        uint4 rk[kRowsPerIter], rv[kRowsPerIter];
#pragma unroll
        for (int r = 0; r < kRowsPerIter; ++r) {
            const int j = j0 + r;
            if (j < r1) {
                const uint4 *pk = (j < len) ? Kcu + (size_t)j * LPR : knu;
                const uint4 *pv = (j < len) ? Vcu + (size_t)j * LPR : vnu;
                rk[r] = ld_row(pk + l);
                rv[r] = ld_row(pv + l);
            } else {
                rk[r] = make_uint4(0, 0, 0, 0);
                rv[r] = make_uint4(0, 0, 0, 0);
            }
        }
        float s[kRowsPerIter];
#pragma unroll
        for (int r = 0; r < kRowsPerIter; ++r) {
            float f[8];
            unpack8(rk[r], f);
            float d = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) d = fmaf(qf[i], f[i], d);
#pragma unroll
            for (int o = LPR / 2; o >= 1; o >>= 1) d += __shfl_xor_sync(gmask, d, o);
            s[r] = (j0 + r < r1) ? d : -INFINITY;
        }
        float mn = m;
#pragma unroll
        for (int r = 0; r < kRowsPerIter; ++r) mn = fmaxf(mn, s[r]);
        const float corr = fast_exp2(m - mn);      // first pass: exp2(-inf) = 0
        m = mn;
        lsum *= corr;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] *= corr;
#pragma unroll
        for (int r = 0; r < kRowsPerIter; ++r) {
            const float p = fast_exp2(s[r] - mn);
            lsum += p;
            float f[8];
            unpack8(rv[r], f);
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = fmaf(p, f[i], acc[i]);
        }
    }

    if (l == 0) { sm_m[g] = m; sm_l[g] = lsum; }
#pragma unroll
    for (int i = 0; i < 8; ++i) sm_acc[g][l * 8 + i] = acc[i];
    __syncthreads();   // also orders every cache read of this CTA before the slot write below

    for (int d = threadIdx.x; d < D; d += kDecThreads) {
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
    if (splits == 1 && threadIdx.x >= kDecThreads - 2 * LPR) {
        const int i = threadIdx.x - (kDecThreads - 2 * LPR);
        if (i < LPR) Kcu[(size_t)write_slot * LPR + i] = knu[i];
        else         Vcu[(size_t)write_slot * LPR + (i - LPR)] = vnu[i - LPR];
    }
}

// Merges the per-split partials of one unit, writes out and stores the new row.
template <int LPR>
__global__ void combine_kernel(const float *__restrict__ partials, int splits,
                               const uint4 *__restrict__ k_new, const uint4 *__restrict__ v_new,
                               uint4 *Kc, uint4 *Vc, int cap, int write_slot, __nv_bfloat16 *__restrict__ out)
{
    constexpr int D = LPR * 8;
    const int unit = blockIdx.x;
    const int d = threadIdx.x;
    const float *p = partials + (size_t)unit * splits * (D + 2);
    if (d < D) {
        float M = -INFINITY;
        for (int s = 0; s < splits; ++s) M = fmaxf(M, p[(size_t)s * (D + 2) + D]);
        float L = 0.f, A = 0.f;
        for (int s = 0; s < splits; ++s) {
            const float ms = p[(size_t)s * (D + 2) + D];
            const float w = (ms == -INFINITY) ? 0.f : fast_exp2(ms - M);
            L = fmaf(p[(size_t)s * (D + 2) + D + 1], w, L);
            A = fmaf(p[(size_t)s * (D + 2) + d], w, A);
        }
        out[(size_t)unit * D + d] = __float2bfloat16_rn(A / L);
    }
    if (d < 2 * LPR) {
        uint4 *Kcu = Kc + (size_t)unit * cap * LPR;
        uint4 *Vcu = Vc + (size_t)unit * cap * LPR;
        if (d < LPR) Kcu[(size_t)write_slot * LPR + d] = k_new[(size_t)unit * LPR + d];
        else         Vcu[(size_t)write_slot * LPR + (d - LPR)] = v_new[(size_t)unit * LPR + (d - LPR)];
    }
}

}  // namespace

// Split the rows of a unit over several CTAs only when there are too few units to fill
// the GPU; every split keeps at least 64 rows.
int decode_splits(int units, int rows)
{
    const int target = 148 * 4;
    int s = (target + units - 1) / units;
    int max_s = (rows + 63) / 64;
    if (s > max_s) s = max_s;
    if (s < 1) s = 1;
    return s;
}

cudaError_t launch_decode(const void *q, const void *k_new, const void *v_new, void *Kc, void *Vc,
                          int units, int D, int cap, int len, int write_slot, float scale, void *out,
                          float *partials, int splits, cudaStream_t stream)
{
    const float sl2 = scale * 1.4426950408889634f;
    const long long grid = (long long)units * splits;
    if (grid > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    if (D == 128) {
        decode_kernel<16><<<(unsigned)grid, kDecThreads, 0, stream>>>(
            (const uint4 *)q, (const uint4 *)k_new, (const uint4 *)v_new, (uint4 *)Kc, (uint4 *)Vc, cap, len,
            write_slot, sl2, (__nv_bfloat16 *)out, partials, splits);
        if (splits > 1)
            combine_kernel<16><<<units, 128, 0, stream>>>(partials, splits, (const uint4 *)k_new,
                                                          (const uint4 *)v_new, (uint4 *)Kc, (uint4 *)Vc, cap,
                                                          write_slot, (__nv_bfloat16 *)out);
    } else {
        decode_kernel<8><<<(unsigned)grid, kDecThreads, 0, stream>>>(
            (const uint4 *)q, (const uint4 *)k_new, (const uint4 *)v_new, (uint4 *)Kc, (uint4 *)Vc, cap, len,
            write_slot, sl2, (__nv_bfloat16 *)out, partials, splits);
        if (splits > 1)
            combine_kernel<8><<<units, 64, 0, stream>>>(partials, splits, (const uint4 *)k_new,
                                                         (const uint4 *)v_new, (uint4 *)Kc, (uint4 *)Vc, cap,
                                                         write_slot, (__nv_bfloat16 *)out);
    }
    return cudaGetLastError();
}

}  // namespace ec
