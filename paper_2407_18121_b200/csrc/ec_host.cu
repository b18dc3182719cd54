// Entry points for callers whose tensors start in host memory: they enqueue the host<->device
// copies around the device calls. Nothing is computed on the host.
#include "ec_common.cuh"

namespace {

struct EventPool {                       // events of one call, destroyed when it returns
    cudaEvent_t ev[64];
    int n = 0;
    cudaEvent_t get()
    {
        if (n >= 64) return nullptr;
        if (cudaEventCreateWithFlags(&ev[n], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        return ev[n++];
    }
    ~EventPool() { for (int i = 0; i < n; ++i) cudaEventDestroy(ev[i]); }
};

}  // namespace

extern "C" {

int ec_compress_host(const void *Q_host, const void *K_host, const void *V_host, void *Q_dev, void *K_dev, void *V_dev,
                     float *scores_dev, int N, int H, int T, int D, float scale, int n_keep, int population,
                     int protect_ends, void *Kc_dev, void *Vc_dev, int cap, int32_t *anchor_pos_dev,
                     int32_t *anchor_pos_host, void *ws_imp, size_t ws_imp_bytes, void *ws_sel, size_t ws_sel_bytes,
                     void *stream)
{
    ec::NvtxRange nvtx_range("ec_compress_host");
    if (!Q_host || !K_host || !V_host || !Q_dev || !K_dev || !V_dev) return EC_ERR_NULL;
    if (N < 1 || H < 1 || T < 1 || (D != 64 && D != 128)) return EC_ERR_SHAPE;
    if (population != EC_PER_HEAD && population != EC_LAYER_SHARED) return EC_ERR_ARG;
    // everything the two device calls would reject is rejected here, before the first copy is enqueued
    int pre = ec::check_importance_args(Q_dev, K_dev, scores_dev, nullptr, N, H, T, D, scale, ws_imp, ws_imp_bytes);
    if (pre != EC_OK) return pre;
    pre = ec::check_select_compact_args(K_dev, V_dev, scores_dev, N, H, T, D, n_keep, population == EC_LAYER_SHARED ? H : 1,
                                        EC_COMPACT_MERGE, Kc_dev, Vc_dev, cap, anchor_pos_dev, nullptr, ws_sel, ws_sel_bytes);
    if (pre != EC_OK) return pre;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t bytes = (size_t)N * H * T * D * 2;
    if (cudaMemcpyAsync(Q_dev, Q_host, bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return EC_ERR_CUDA;
    if (cudaMemcpyAsync(K_dev, K_host, bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return EC_ERR_CUDA;
    if (cudaMemcpyAsync(V_dev, V_host, bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return EC_ERR_CUDA;
    int st = ec_importance(Q_dev, K_dev, scores_dev, nullptr, N, H, T, D, scale, ws_imp, ws_imp_bytes, stream);
    if (st != EC_OK) return st;
    st = ec_select_merge(K_dev, V_dev, scores_dev, N, H, T, D, n_keep, population, protect_ends, Kc_dev, Vc_dev, cap,
                         anchor_pos_dev, nullptr, ws_sel, ws_sel_bytes, stream);
    if (st != EC_OK) return st;
    if (anchor_pos_host &&
        cudaMemcpyAsync(anchor_pos_host, anchor_pos_dev, (size_t)N * H * n_keep * sizeof(int32_t), cudaMemcpyDeviceToHost,
                        s) != cudaSuccess)
        return EC_ERR_CUDA;
    return EC_OK;
}

int ec_decode_steps_host(const void *q_host, const void *k_host, const void *v_host, void *out_host, void *q_dev,
                         void *k_dev, void *v_dev, void *out_dev, int steps, int chunk, ec_cache *c, float scale,
                         void *ws, size_t ws_bytes, void *stream, void *upload_stream, void *download_stream)
{
    ec::NvtxRange nvtx_range("ec_decode_steps_host");
    if (!q_host || !k_host || !v_host || !out_host || !q_dev || !k_dev || !v_dev || !out_dev || !c) return EC_ERR_NULL;
    if (!upload_stream || !download_stream) return EC_ERR_NULL;
    if (steps < 0 || chunk < 1) return EC_ERR_ARG;
    // the cache struct, the scalar arguments and the workspace are checked before anything is enqueued;
    // what can still fail later is a CUDA runtime call or, under the retention-ratio policy, a cache
    // that has no room left to grow: c->step then tells how many steps were taken
    int pre = ec::check_cache(c);
    if (pre != EC_OK) return pre;
    if (!(scale > 0.f) || !(scale < 3.0e38f)) return EC_ERR_ARG;
    if (!ws || ws_bytes < ec_decode_workspace(c)) return EC_ERR_WORKSPACE;
    if (((uintptr_t)ws & 255u) || ((uintptr_t)q_dev & 15u) || ((uintptr_t)k_dev & 15u) || ((uintptr_t)v_dev & 15u) ||
        ((uintptr_t)out_dev & 15u))
        return EC_ERR_ALIGN;
    if (steps == 0) return EC_OK;
    const int nchunks = (steps + chunk - 1) / chunk;
    if (2 * nchunks + 2 > 64) return EC_ERR_ARG;                       // at most 31 chunks per call
    cudaStream_t cur = (cudaStream_t)stream, up = (cudaStream_t)upload_stream, down = (cudaStream_t)download_stream;
    const size_t step_bytes = (size_t)c->N * c->H * c->D * 2;
    EventPool pool;
    // the staging buffers may still be in use by earlier work on `stream`
    cudaEvent_t start = pool.get();
    if (!start || cudaEventRecord(start, cur) != cudaSuccess) return EC_ERR_CUDA;
    if (cudaStreamWaitEvent(up, start, 0) != cudaSuccess || cudaStreamWaitEvent(down, start, 0) != cudaSuccess)
        return EC_ERR_CUDA;
    cudaEvent_t ready[31];
    for (int i = 0; i < nchunks; ++i) {
        const size_t off = (size_t)i * chunk * step_bytes;
        const size_t n = (size_t)((i + 1) * chunk <= steps ? chunk : steps - i * chunk) * step_bytes;
        if (cudaMemcpyAsync((char *)q_dev + off, (const char *)q_host + off, n, cudaMemcpyHostToDevice, up) != cudaSuccess ||
            cudaMemcpyAsync((char *)k_dev + off, (const char *)k_host + off, n, cudaMemcpyHostToDevice, up) != cudaSuccess ||
            cudaMemcpyAsync((char *)v_dev + off, (const char *)v_host + off, n, cudaMemcpyHostToDevice, up) != cudaSuccess)
            return EC_ERR_CUDA;
        ready[i] = pool.get();
        if (!ready[i] || cudaEventRecord(ready[i], up) != cudaSuccess) return EC_ERR_CUDA;
    }
    for (int i = 0; i < nchunks; ++i) {
        const size_t off = (size_t)i * chunk * step_bytes;
        const int ns = (i + 1) * chunk <= steps ? chunk : steps - i * chunk;
        if (cudaStreamWaitEvent(cur, ready[i], 0) != cudaSuccess) return EC_ERR_CUDA;
        int st = ec_decode_steps((char *)q_dev + off, (char *)k_dev + off, (char *)v_dev + off, ns, c, scale,
                                 (char *)out_dev + off, nullptr, ws, ws_bytes, stream);
        if (st != EC_OK) return st;
        cudaEvent_t done = pool.get();
        if (!done || cudaEventRecord(done, cur) != cudaSuccess || cudaStreamWaitEvent(down, done, 0) != cudaSuccess)
            return EC_ERR_CUDA;
        if (cudaMemcpyAsync((char *)out_host + off, (char *)out_dev + off, (size_t)ns * step_bytes, cudaMemcpyDeviceToHost,
                            down) != cudaSuccess)
            return EC_ERR_CUDA;
    }
    cudaEvent_t fin = pool.get();
    if (!fin || cudaEventRecord(fin, down) != cudaSuccess || cudaStreamWaitEvent(cur, fin, 0) != cudaSuccess)
        return EC_ERR_CUDA;
    return EC_OK;
}

}  // extern "C"
