// Measurement aids that sit beside the method's kernels: a read-only streaming kernel whose
// achieved rate is the ceiling a read-dominated kernel (decode attention, merge) can be held
// against, and a query of the decode launch shape.
#include "ec_common.cuh"

namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbeUnroll = 8;
constexpr size_t kProbeChunk = (size_t)kProbeThreads * kProbeUnroll;   // 16-byte vectors per CTA: 32 KB

// One CTA per contiguous 32 KB chunk, eight independent 16-byte loads in flight per thread, the
// hardware scheduler refilling SMs as CTAs retire. Of the shapes tried on B200 over 4 GiB (grid-stride
// and chunked persistent grids of 4-32 CTAs per SM, 64-512 threads, 4-16 loads per thread: 6.7-7.4
// TB/s) this one read fastest (7.47 TB/s). What is read is folded into one word so that no load
// can be dropped.
// write_every > 0: of every `write_every` consecutive 256-byte rows read, the first is also
// written to `dst` (densely), which gives the read/write mix of a merge at keep ratio
// 1/write_every; 0: nothing is written.
__global__ void __launch_bounds__(kProbeThreads)
read_stream_kernel(const uint4 *__restrict__ buf, size_t n_vec, uint4 *__restrict__ dst, int write_every,
                   unsigned *__restrict__ sink)
{
    const size_t base = (size_t)blockIdx.x * kProbeChunk + threadIdx.x;
    unsigned acc = 0;
    auto maybe_write = [&](size_t i, const uint4 &v) {
        const size_t row = i >> 4;                                      // 16 vectors = one 256-byte row
        if (write_every > 0 && row % (size_t)write_every == 0) dst[(row / (size_t)write_every) * 16 + (i & 15)] = v;
    };
    if (base - threadIdx.x + kProbeChunk <= n_vec) {
        uint4 v[kProbeUnroll];
#pragma unroll
        for (int j = 0; j < kProbeUnroll; ++j) v[j] = ec::ldg_stream(buf + base + (size_t)j * kProbeThreads);
#pragma unroll
        for (int j = 0; j < kProbeUnroll; ++j) {
            acc ^= v[j].x ^ v[j].y ^ v[j].z ^ v[j].w;
            maybe_write(base + (size_t)j * kProbeThreads, v[j]);
        }
    } else {
        for (size_t i = base; i < n_vec; i += kProbeThreads) {          // the ragged last chunk
            const uint4 v = ec::ldg_stream(buf + i);
            acc ^= v.x ^ v.y ^ v.z ^ v.w;
            maybe_write(i, v);
        }
    }
    acc = __reduce_xor_sync(0xFFFFFFFFu, acc);
    if ((threadIdx.x & 31) == 0 && acc != 0) atomicXor(sink, acc);
}

}  // namespace

extern "C" {

int ec_probe_read_stream(const void *buf, size_t bytes, unsigned *sink, void *stream)
{
    return ec_probe_mixed_stream(buf, bytes, nullptr, 0, sink, stream);
}

int ec_probe_mixed_stream(const void *buf, size_t bytes, void *dst, int write_every, unsigned *sink, void *stream)
{
    if (!buf || !sink || (write_every > 0 && !dst)) return EC_ERR_NULL;
    if (((uintptr_t)buf & 15u) || ((uintptr_t)sink & 3u) || ((uintptr_t)dst & 15u)) return EC_ERR_ALIGN;
    if (bytes < 16 || (bytes & 15u) || write_every < 0) return EC_ERR_ARG;
    const size_t n_vec = bytes / 16;
    const size_t ctas = (n_vec + kProbeChunk - 1) / kProbeChunk;
    if (ctas > 0x7FFFFFFFull) return EC_ERR_ARG;                  // at most 64 TiB per call
    const unsigned grid = (unsigned)ctas;
    read_stream_kernel<<<grid, kProbeThreads, 0, (cudaStream_t)stream>>>((const uint4 *)buf, n_vec, (uint4 *)dst, write_every,
                                                                          sink);
    return cudaGetLastError() == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

int ec_decode_splits(const ec_cache *c)
{
    if (ec::check_cache(c) != EC_OK) return 0;
    return ec::decode_splits(c->N * c->H, c->len + 1);
}

}  // extern "C"
