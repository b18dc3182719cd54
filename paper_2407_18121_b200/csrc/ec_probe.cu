// Measurement aids that sit beside the method's kernels: a read-only streaming kernel whose
// achieved rate is the ceiling a read-dominated kernel (decode attention, merge) can be held
// against, and a query of the decode launch shape.
#include "ec_common.cuh"

namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbeUnroll = 8;

// Every CTA walks the buffer with a grid-wide stride, kProbeUnroll independent 16-byte loads in
// flight per thread, and folds what it read into one word so that no load can be dropped.
__global__ void __launch_bounds__(kProbeThreads)
read_stream_kernel(const uint4 *__restrict__ buf, size_t n_vec, unsigned *__restrict__ sink)
{
    const size_t stride = (size_t)gridDim.x * kProbeThreads;
    size_t i = (size_t)blockIdx.x * kProbeThreads + threadIdx.x;
    unsigned acc = 0;
    for (; i + (kProbeUnroll - 1) * stride < n_vec; i += kProbeUnroll * stride) {
        uint4 v[kProbeUnroll];
#pragma unroll
        for (int j = 0; j < kProbeUnroll; ++j) v[j] = ec::ldg_stream(buf + i + j * stride);
#pragma unroll
        for (int j = 0; j < kProbeUnroll; ++j) acc ^= v[j].x ^ v[j].y ^ v[j].z ^ v[j].w;
    }
    for (; i < n_vec; i += stride) {
        const uint4 v = ec::ldg_stream(buf + i);
        acc ^= v.x ^ v.y ^ v.z ^ v.w;
    }
    acc = __reduce_xor_sync(0xFFFFFFFFu, acc);
    if ((threadIdx.x & 31) == 0 && acc != 0) atomicXor(sink, acc);
}

}  // namespace

extern "C" {

int ec_probe_read_stream(const void *buf, size_t bytes, unsigned *sink, void *stream)
{
    if (!buf || !sink) return EC_ERR_NULL;
    if (((uintptr_t)buf & 15u) || ((uintptr_t)sink & 3u)) return EC_ERR_ALIGN;
    if (bytes < 16 || (bytes & 15u)) return EC_ERR_ARG;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return EC_ERR_CUDA;
    const size_t n_vec = bytes / 16;
    size_t want = (n_vec + kProbeThreads - 1) / kProbeThreads;
    const size_t resident = (size_t)sms * 8;                 // eight 256-thread CTAs per SM
    const unsigned grid = (unsigned)(want < resident ? want : resident);
    read_stream_kernel<<<grid, kProbeThreads, 0, (cudaStream_t)stream>>>((const uint4 *)buf, n_vec, sink);
    return cudaGetLastError() == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

int ec_decode_splits(const ec_cache *c)
{
    if (ec::check_cache(c) != EC_OK) return 0;
    return ec::decode_splits(c->N * c->H, c->len + 1);
}

}  // extern "C"
