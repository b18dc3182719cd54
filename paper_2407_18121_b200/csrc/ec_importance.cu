// Importance of every prompt key (Sec. 3.3, Eq. 1 and the column sums that follow it),
// computed in two passes so that the T x T attention matrix is never stored:
//   pass 1: lse[m]   = log sum_{n<=m} exp(scale*<q_m,k_n>)
//   pass 2: score[n] = sum_{m>=n} exp(scale*<q_m,k_n> - lse[m])
#include "ec_common.cuh"

namespace ec {

namespace {

constexpr int kTile = 32;
constexpr float kLog2e = 1.4426950408889634f;

// Loads `kTile` bf16 rows starting at row0 into fp32 shared memory (rows past T -> 0).
template <int D>
__device__ __forceinline__ void load_tile(const __nv_bfloat16 *__restrict__ X, int row0, int T,
                                          float (*dst)[D + 1], int tid)
{
    for (int e = tid; e < kTile * D; e += kTile * kTile) {
        int r = e / D, c = e - r * D;
        int row = row0 + r;
        dst[r][c] = (row < T) ? __bfloat162float(X[(size_t)row * D + c]) : 0.f;
    }
}

template <int D>
__device__ __forceinline__ float dot_rows(const float (*A)[D + 1], int a, const float (*B)[D + 1], int b)
{
    float acc = 0.f;
#pragma unroll 16
    for (int c = 0; c < D; ++c) acc = fmaf(A[a][c], B[b][c], acc);
    return acc;
}

// grid = (units, query tiles); block = 32 x 32: thread (ty = query, tx = key).
template <int D>
__global__ void __launch_bounds__(kTile * kTile)
lse_kernel(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K, int T, float scale_log2e,
           float *__restrict__ lse2 /* log2 domain, workspace */, float *__restrict__ lse_out /* natural, optional */)
{
    __shared__ float Qs[kTile][D + 1];
    __shared__ float Ks[kTile][D + 1];
    const int tx = threadIdx.x, ty = threadIdx.y, tid = ty * kTile + tx;
    const size_t unit = blockIdx.x;
    const int m0 = blockIdx.y * kTile;
    const __nv_bfloat16 *Qu = Q + unit * T * D, *Ku = K + unit * T * D;
    load_tile<D>(Qu, m0, T, Qs, tid);
    const int m = m0 + ty;
    float M = -INFINITY, Z = 0.f;
    for (int n0 = 0; n0 <= m0; n0 += kTile) {
        __syncthreads();
        load_tile<D>(Ku, n0, T, Ks, tid);
        __syncthreads();
        const int n = n0 + tx;
        float s = dot_rows<D>(Qs, ty, Ks, tx) * scale_log2e;
        if (n > m || m >= T) s = -INFINITY;
        float mx = s;
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        const float Mn = fmaxf(M, mx);
        float p = (s == -INFINITY) ? 0.f : exp2f(s - Mn);
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) p += __shfl_xor_sync(0xFFFFFFFFu, p, o);
        if (Mn != -INFINITY) { Z = Z * exp2f(M - Mn) + p; M = Mn; }
    }
    if (tx == 0 && m < T) {
        const float l2 = M + log2f(Z);
        lse2[unit * T + m] = l2;
        if (lse_out) lse_out[unit * T + m] = l2 * 0.6931471805599453f;
    }
}

// grid = (units, key tiles); block = 32 x 32: thread (ty = key, tx = query).
template <int D>
__global__ void __launch_bounds__(kTile * kTile)
colsum_kernel(const __nv_bfloat16 *__restrict__ Q, const __nv_bfloat16 *__restrict__ K, int T, float scale_log2e,
              const float *__restrict__ lse2, float *__restrict__ scores)
{
    __shared__ float Ks[kTile][D + 1];
    __shared__ float Qs[kTile][D + 1];
    const int tx = threadIdx.x, ty = threadIdx.y, tid = ty * kTile + tx;
    const size_t unit = blockIdx.x;
    const int n0 = blockIdx.y * kTile;
    const __nv_bfloat16 *Qu = Q + unit * T * D, *Ku = K + unit * T * D;
    load_tile<D>(Ku, n0, T, Ks, tid);
    const int n = n0 + ty;
    float acc = 0.f;
    for (int m0 = n0; m0 < T; m0 += kTile) {
        __syncthreads();
        load_tile<D>(Qu, m0, T, Qs, tid);
        __syncthreads();
        const int m = m0 + tx;
        float p = 0.f;
        if (m < T && m >= n) {
            const float s = dot_rows<D>(Ks, ty, Qs, tx) * scale_log2e;
            p = exp2f(s - lse2[unit * T + m]);
        }
#pragma unroll
        for (int o = 16; o >= 1; o >>= 1) p += __shfl_xor_sync(0xFFFFFFFFu, p, o);
        acc += p;
    }
    if (tx == 0 && n < T) scores[unit * T + n] = acc;
}

}  // namespace

size_t importance_workspace_bytes(int N, int H, int T, int D)
{
    (void)D;
    size_t lse = (size_t)N * H * T * sizeof(float);
    return kStatusBytes + ((lse + 255) / 256) * 256;
}

cudaError_t launch_importance(const void *Q, const void *K, float *scores, float *lse_out,
                              int N, int H, int T, int D, float scale, void *ws, cudaStream_t stream)
{
    cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, stream);
    if (e != cudaSuccess) return e;
    float *lse2 = reinterpret_cast<float *>(static_cast<char *>(ws) + kStatusBytes);
    const int units = N * H;
    dim3 block(kTile, kTile);
    dim3 grid(units, (T + kTile - 1) / kTile);
    const float sl2 = scale * kLog2e;
    const __nv_bfloat16 *q = (const __nv_bfloat16 *)Q, *k = (const __nv_bfloat16 *)K;
    if (D == 128) {
        lse_kernel<128><<<grid, block, 0, stream>>>(q, k, T, sl2, lse2, lse_out);
        colsum_kernel<128><<<grid, block, 0, stream>>>(q, k, T, sl2, lse2, scores);
    } else {
        lse_kernel<64><<<grid, block, 0, stream>>>(q, k, T, sl2, lse2, lse_out);
        colsum_kernel<64><<<grid, block, 0, stream>>>(q, k, T, sl2, lse2, scores);
    }
    return cudaGetLastError();
}

}  // namespace ec
