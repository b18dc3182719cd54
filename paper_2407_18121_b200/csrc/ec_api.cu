// C ABI of the library: argument validation, workspace layout and kernel sequencing.
// Every step of the path runs in the CUDA kernels; nothing here computes on the host
// beyond integer bookkeeping of the cache (which slot the next row goes to).
#include "ec_common.cuh"

#include <math.h>

namespace {

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline size_t round256(size_t x) { return (x + 255) / 256 * 256; }

constexpr int kMaxT = 16384;

int check_shape(int N, int H, int T, int D)
{
    if (N < 1 || H < 1 || T < 1 || T > kMaxT) return EC_ERR_SHAPE;
    if (D != 64 && D != 128) return EC_ERR_SHAPE;
    if ((long long)N * H * T >= (1LL << 31)) return EC_ERR_SHAPE;
    if ((long long)N * H >= (1LL << 24)) return EC_ERR_SHAPE;
    return EC_OK;
}

}  // namespace

namespace ec {

// Host-only argument checks, shared by the device-tensor calls and the host-tensor calls (which
// run them before their first copy, so that a rejected call has enqueued nothing).
int check_importance_args(const void *Q, const void *K, const float *scores, const float *lse, int N, int H, int T, int D,
                          float scale, const void *ws, size_t ws_bytes)
{
    if (!Q || !K || !scores) return EC_ERR_NULL;
    int st = check_shape(N, H, T, D);
    if (st != EC_OK) return st;
    if (!(scale > 0.f) || !isfinite(scale)) return EC_ERR_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(scores, 16) || (lse && !aligned(lse, 16))) return EC_ERR_ALIGN;
    if (!ws || ws_bytes < importance_workspace_bytes(N, H, T, D)) return EC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EC_ERR_ALIGN;
    return EC_OK;
}

int check_select_compact_args(const void *K, const void *V, const float *scores, int N, int H, int T, int D, int n_keep,
                              int share, int compaction, const void *Kc, const void *Vc, int cap,
                              const int32_t *anchor_pos, const int32_t *bucket_len, const void *ws, size_t ws_bytes)
{
    if (!K || !V || !scores || !Kc || !Vc || !anchor_pos) return EC_ERR_NULL;
    int st = check_shape(N, H, T, D);
    if (st != EC_OK) return st;
    if (n_keep < 1 || n_keep > T || cap < n_keep) return EC_ERR_ARG;
    if (share < 1 || ((long long)N * H) % share != 0) return EC_ERR_ARG;
    if (compaction != EC_COMPACT_MERGE && compaction != EC_COMPACT_EVICT) return EC_ERR_ARG;
    if ((long long)N * H * cap >= (1LL << 31)) return EC_ERR_SHAPE;
    if (!aligned(K, 16) || !aligned(V, 16) || !aligned(Kc, 16) || !aligned(Vc, 16) || !aligned(scores, 4) ||
        !aligned(anchor_pos, 4) || (bucket_len && !aligned(bucket_len, 4)))
        return EC_ERR_ALIGN;
    if (!ws || ws_bytes < ec_select_compact_workspace(N, H, T, D, n_keep, share)) return EC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EC_ERR_ALIGN;
    return EC_OK;
}

// The caller owns the ec_cache struct and may have filled or restored it by hand: every call that
// reads one repeats the checks of ec_cache_init / ec_cache_init_ratio.
int check_cache(const ec_cache *c)
{
    if (!c) return EC_ERR_NULL;
    if (!c->Kc || !c->Vc) return EC_ERR_NULL;
    if (c->N < 1 || c->H < 1 || (c->D != 64 && c->D != 128) || c->cap < 1) return EC_ERR_SHAPE;
    if ((long long)c->N * c->H * c->cap >= (1LL << 31) || (long long)c->N * c->H >= (1LL << 24)) return EC_ERR_SHAPE;
    if (!aligned(c->Kc, 16) || !aligned(c->Vc, 16)) return EC_ERR_ALIGN;
    if (c->policy == EC_POLICY_RATIO) {
        if (!c->recent_slots_host) return EC_ERR_NULL;
        if (c->offset < 1 || c->len < c->offset || c->len > c->cap || c->recent_head < 0 ||
            c->recent_head >= c->offset || !(c->keep_ratio > 0.0 && c->keep_ratio <= 1.0) || c->n_tot < c->len)
            return EC_ERR_ARG;
    } else if (c->policy == EC_POLICY_FIXED) {
        if (c->budget < 2 || c->budget > c->cap || c->len < 0 || c->len > c->budget || c->offset < 1 ||
            c->offset > c->budget - 1 || c->ring_head < 0 || c->ring_head >= c->offset)
            return EC_ERR_ARG;
    } else {
        return EC_ERR_ARG;
    }
    return EC_OK;
}

}  // namespace ec

extern "C" {

const char *ec_status_string(int status)
{
    switch (status) {
    case EC_OK: return "ok";
    case EC_ERR_NULL: return "required pointer is NULL";
    case EC_ERR_SHAPE: return "unsupported shape";
    case EC_ERR_ALIGN: return "pointer not sufficiently aligned";
    case EC_ERR_ARG: return "argument out of range";
    case EC_ERR_WORKSPACE: return "workspace missing or too small";
    case EC_ERR_CUDA: return "CUDA runtime error";
    case EC_ERR_TIMEOUT: return "device-side wait timed out";
    case EC_ERR_TOO_LARGE: return "problem too large for the built-in scratch";
    default: return "unknown status";
    }
}

int ec_keep_count(int T, double keep_ratio)
{
    if (T < 1 || !(keep_ratio >= 0.0 && keep_ratio <= 1.0)) return 0;
    // Algorithm 1: del_num = int(seq_len - n * retained_fraction) with n = seq_len = T
    int del = (int)((double)T - (double)T * keep_ratio);
    if (del < 0) del = 0;
    int keep = T - del;
    if (keep < 1) keep = 1;
    if (keep > T) keep = T;
    return keep;
}

size_t ec_importance_workspace(int N, int H, int T, int D)
{
    if (check_shape(N, H, T, D) != EC_OK) return 0;
    return ec::importance_workspace_bytes(N, H, T, D);
}

int ec_importance(const void *Q, const void *K, float *scores, float *lse, int N, int H, int T, int D,
                  float scale, void *ws, size_t ws_bytes, void *stream)
{
    ec::NvtxRange nvtx_range("ec_importance");
    int st = ec::check_importance_args(Q, K, scores, lse, N, H, T, D, scale, ws, ws_bytes);
    if (st != EC_OK) return st;
    cudaError_t e = ec::launch_importance(Q, K, scores, lse, nullptr, N, H, T, 0, D, scale, EC_STAT_SUM, 0.0, ws,
                                          (cudaStream_t)stream);
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

int ec_importance_statistic(const void *Q, const void *K, float *scores, float *lse, int N, int H, int Tq, int P, int D,
                            float scale, int statistic, double beta, void *ws, size_t ws_bytes, void *stream)
{
    ec::NvtxRange nvtx_range("ec_importance_statistic");
    if (!Q || !K || !scores) return EC_ERR_NULL;
    if (P < 0 || Tq < 1 || (long long)P + Tq > kMaxT) return EC_ERR_SHAPE;
    int st = check_shape(N, H, Tq + P, D);
    if (st != EC_OK) return st;
    if (!(scale > 0.f) || !isfinite(scale)) return EC_ERR_ARG;
    if (statistic < EC_STAT_SUM || statistic > EC_STAT_MOVING_AVERAGE) return EC_ERR_ARG;
    if (statistic == EC_STAT_MOVING_AVERAGE && !(beta > 0.0 && beta < 1.0)) return EC_ERR_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(scores, 16) || (lse && !aligned(lse, 16))) return EC_ERR_ALIGN;
    if (!ws || ws_bytes < ec::importance_workspace_bytes(N, H, Tq, D)) return EC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EC_ERR_ALIGN;
    cudaError_t e = ec::launch_importance(Q, K, scores, lse, nullptr, N, H, Tq, P, D, scale, statistic, beta, ws,
                                          (cudaStream_t)stream);
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

int ec_importance_prefix(const void *Q, const void *K, float *scores, float *lse, int N, int H, int Tq, int P, int D,
                         float scale, void *ws, size_t ws_bytes, void *stream)
{
    return ec_importance_statistic(Q, K, scores, lse, N, H, Tq, P, D, scale, EC_STAT_SUM, 0.0, ws, ws_bytes, stream);
}

int ec_importance_from_lse(const void *Q, const void *K, const float *lse, float *scores, int N, int H, int T, int D,
                           float scale, void *ws, size_t ws_bytes, void *stream)
{
    ec::NvtxRange nvtx_range("ec_importance_from_lse");
    if (!Q || !K || !scores || !lse) return EC_ERR_NULL;
    int st = check_shape(N, H, T, D);
    if (st != EC_OK) return st;
    if (!(scale > 0.f) || !isfinite(scale)) return EC_ERR_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(scores, 16) || !aligned(lse, 4)) return EC_ERR_ALIGN;
    if (!ws || ws_bytes < ec::importance_workspace_bytes(N, H, T, D)) return EC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EC_ERR_ALIGN;
    cudaError_t e = ec::launch_importance(Q, K, scores, nullptr, lse, N, H, T, 0, D, scale, EC_STAT_SUM, 0.0, ws,
                                          (cudaStream_t)stream);
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

int ec_prefill_attention(const void *Q, const void *K, const void *V, void *out, float *lse, float *scores, int N, int H,
                         int Tq, int P, int D, float scale, void *ws, size_t ws_bytes, void *stream)
{
    ec::NvtxRange nvtx_range("ec_prefill_attention");
    if (!Q || !K || !V || !out) return EC_ERR_NULL;
    if (P < 0 || Tq < 1 || (long long)P + Tq > kMaxT) return EC_ERR_SHAPE;
    int st = check_shape(N, H, Tq + P, D);
    if (st != EC_OK) return st;
    if (!(scale > 0.f) || !isfinite(scale)) return EC_ERR_ARG;
    if (!aligned(Q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(out, 16) || (lse && !aligned(lse, 16)) ||
        (scores && !aligned(scores, 16)))
        return EC_ERR_ALIGN;
    if (!ws || ws_bytes < ec::importance_workspace_bytes(N, H, Tq, D)) return EC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EC_ERR_ALIGN;
    cudaError_t e = ec::launch_attention(Q, K, V, out, lse, N, H, Tq, P, D, scale, ws, (cudaStream_t)stream);
    if (e == cudaSuccess && scores)
        e = ec::launch_importance(Q, K, scores, nullptr, ec::kLseInWorkspace, N, H, Tq, P, D, scale, EC_STAT_SUM, 0.0, ws,
                                  (cudaStream_t)stream);
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

int ec_selftest_wait_timeout(void *ws, unsigned limit_us, void *stream)
{
    if (!ws) return EC_ERR_NULL;
    if (!aligned(ws, 256)) return EC_ERR_ALIGN;
    if (limit_us < 1 || limit_us > 1000000u) return EC_ERR_ARG;
    return ec::launch_wait_selftest(ws, limit_us, (cudaStream_t)stream) == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

int ec_device_status(void *ws, void *stream)
{
    if (!ws) return EC_ERR_NULL;
    int word = 0;
    cudaError_t e = cudaMemcpyAsync(&word, ws, sizeof word, cudaMemcpyDeviceToHost, (cudaStream_t)stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return EC_ERR_CUDA;
    return word == 0 ? EC_OK : EC_ERR_TIMEOUT;
}

size_t ec_select_compact_workspace(int N, int H, int T, int D, int n_keep, int share)
{
    if (check_shape(N, H, T, D) != EC_OK || n_keep < 1 || n_keep > T) return 0;
    if (share < 1 || ((long long)N * H) % share != 0) return 0;
    // a shared population keeps the averaged scores [N*H/share, T]; a minimum keeps the pointer non-null
    size_t mean = (share > 1) ? round256((size_t)N * H / share * T * sizeof(float)) : 0;
    return 256 + mean;
}

int ec_select_compact(const void *K, const void *V, const float *scores, int N, int H, int T, int D, int n_keep,
                      int share, int protect_ends, int compaction, void *Kc, void *Vc, int cap, int32_t *anchor_pos,
                      int32_t *bucket_len, void *ws, size_t ws_bytes, void *stream)
{
    ec::NvtxRange nvtx_range("ec_select_compact");
    int st = ec::check_select_compact_args(K, V, scores, N, H, T, D, n_keep, share, compaction, Kc, Vc, cap, anchor_pos,
                                           bucket_len, ws, ws_bytes);
    if (st != EC_OK) return st;
    float *mean_ws = reinterpret_cast<float *>(static_cast<char *>(ws) + 256);
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = ec::launch_select(scores, N * H, T, n_keep, share, protect_ends ? 1 : 0, anchor_pos, bucket_len,
                                      mean_ws, s);
    if (e != cudaSuccess) return EC_ERR_CUDA;
    if (compaction == EC_COMPACT_MERGE) e = ec::launch_merge(K, V, anchor_pos, N * H, T, D, n_keep, Kc, Vc, cap, s);
    else e = ec::launch_gather(K, V, anchor_pos, N * H, T, D, n_keep, Kc, Vc, cap, s);
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

size_t ec_select_merge_workspace(int N, int H, int T, int D, int n_keep, int population)
{
    return ec_select_compact_workspace(N, H, T, D, n_keep, population == EC_LAYER_SHARED ? H : 1);
}

int ec_select_merge(const void *K, const void *V, const float *scores, int N, int H, int T, int D, int n_keep,
                    int population, int protect_ends, void *Kc, void *Vc, int cap, int32_t *anchor_pos,
                    int32_t *bucket_len, void *ws, size_t ws_bytes, void *stream)
{
    if (population != EC_PER_HEAD && population != EC_LAYER_SHARED) return EC_ERR_ARG;
    return ec_select_compact(K, V, scores, N, H, T, D, n_keep, population == EC_LAYER_SHARED ? H : 1, protect_ends,
                             EC_COMPACT_MERGE, Kc, Vc, cap, anchor_pos, bucket_len, ws, ws_bytes, stream);
}

int ec_cache_init(ec_cache *c, void *Kc, void *Vc, int N, int H, int D, int cap, int len, int budget, int offset)
{
    if (!c || !Kc || !Vc) return EC_ERR_NULL;
    if (N < 1 || H < 1 || (D != 64 && D != 128) || cap < 1) return EC_ERR_SHAPE;
    if ((long long)N * H * cap >= (1LL << 31) || (long long)N * H >= (1LL << 24)) return EC_ERR_SHAPE;
    if (!aligned(Kc, 16) || !aligned(Vc, 16)) return EC_ERR_ALIGN;
    if (budget < 2 || budget > cap || len < 0 || len > budget) return EC_ERR_ARG;
    if (offset < 1 || offset > budget - 1) return EC_ERR_ARG;
    c->Kc = Kc; c->Vc = Vc;
    c->N = N; c->H = H; c->D = D; c->cap = cap;
    c->len = len; c->budget = budget; c->offset = offset;
    c->ring_head = 0;
    c->step = 0;
    c->policy = EC_POLICY_FIXED;
    c->recent_head = 0;
    c->keep_ratio = 0.0;
    c->n_tot = 0;
    c->recent_slots_host = nullptr;
    c->queue_slots_host = nullptr;
    return EC_OK;
}

int ec_cache_concat(const ec_cache *c, const void *K_new, const void *V_new, int Tq, void *K_all, void *V_all,
                    void *stream)
{
    ec::NvtxRange nvtx_range("ec_cache_concat");
    if (!c || !K_new || !V_new || !K_all || !V_all) return EC_ERR_NULL;
    int st = ec::check_cache(c);
    if (st != EC_OK) return st;
    if (c->policy == EC_POLICY_RATIO && !c->queue_slots_host) return EC_ERR_ARG;   // order not tracked
    if (Tq < 1 || c->len < 1) return EC_ERR_ARG;
    const long long units = (long long)c->N * c->H;
    if (units * ((long long)c->len + Tq) >= (1LL << 31)) return EC_ERR_SHAPE;
    if (!aligned(K_new, 16) || !aligned(V_new, 16) || !aligned(K_all, 16) || !aligned(V_all, 16)) return EC_ERR_ALIGN;
    cudaError_t e;
    if (c->policy == EC_POLICY_RATIO) {
        for (int j = 0; j < c->len; ++j)
            if (c->queue_slots_host[j] < 0 || c->queue_slots_host[j] >= c->cap) return EC_ERR_ARG;
        e = ec::launch_concat_listed(c->Kc, c->Vc, (int)units, c->cap, c->D, c->len, c->queue_slots_host, K_new, V_new, Tq,
                                     K_all, V_all, (cudaStream_t)stream);
    } else {
        const bool full = c->len == c->budget;           // the ring exists once the cache has reached its budget
        e = ec::launch_concat(c->Kc, c->Vc, (int)units, c->cap, c->D, c->len, full ? c->budget - c->offset : c->len,
                              full ? c->offset : 0, full ? c->ring_head : 0, K_new, V_new, Tq, K_all, V_all,
                              (cudaStream_t)stream);
    }
    return e == cudaSuccess ? EC_OK : EC_ERR_CUDA;
}

int ec_cache_init_ratio(ec_cache *c, void *Kc, void *Vc, int N, int H, int D, int cap, int len, int offset,
                        double keep_ratio, int64_t n_tot, int *recent_slots)
{
    if (!c || !Kc || !Vc || !recent_slots) return EC_ERR_NULL;
    if (N < 1 || H < 1 || (D != 64 && D != 128) || cap < 1) return EC_ERR_SHAPE;
    if ((long long)N * H * cap >= (1LL << 31) || (long long)N * H >= (1LL << 24)) return EC_ERR_SHAPE;
    if (!aligned(Kc, 16) || !aligned(Vc, 16)) return EC_ERR_ALIGN;
    if (offset < 1 || len < offset || len > cap) return EC_ERR_ARG;
    if (!(keep_ratio > 0.0 && keep_ratio <= 1.0) || n_tot < len) return EC_ERR_ARG;
    c->Kc = Kc; c->Vc = Vc;
    c->N = N; c->H = H; c->D = D; c->cap = cap;
    c->len = len; c->budget = len; c->offset = offset;
    c->ring_head = 0;
    c->step = 0;
    c->policy = EC_POLICY_RATIO;
    c->recent_head = 0;
    c->keep_ratio = keep_ratio;
    c->n_tot = n_tot;
    c->recent_slots_host = recent_slots;
    c->queue_slots_host = nullptr;
    for (int i = 0; i < offset; ++i) recent_slots[i] = len - offset + i;   // oldest first
    return EC_OK;
}

int ec_cache_track_order(ec_cache *c, int *queue_slots)
{
    if (!c || !queue_slots) return EC_ERR_NULL;
    int st = ec::check_cache(c);
    if (st != EC_OK) return st;
    if (c->policy != EC_POLICY_RATIO || c->step != 0) return EC_ERR_ARG;
    for (int i = 0; i < c->len; ++i) queue_slots[i] = i;
    c->queue_slots_host = queue_slots;
    return EC_OK;
}

size_t ec_decode_workspace(const ec_cache *c)
{
    // shape fields only: the query is also made on a struct whose rows are not set up yet
    if (!c || c->N < 1 || c->H < 1 || (c->D != 64 && c->D != 128) || c->cap < 1) return 0;
    if ((long long)c->N * c->H >= (1LL << 24)) return 0;
    const int units = c->N * c->H;
    const int splits = ec::decode_splits(units, c->cap + 1);
    // arrival counters (one int per unit) followed by the per-split partial results
    return round256((size_t)units * sizeof(int)) + round256((size_t)units * splits * (c->D + 2) * sizeof(float));
}

}  // extern "C"

namespace {

// One decode step. `fresh_ws`: nothing is known about the workspace's contents, so the arrival
// counters are cleared first (later steps of a native loop find them cleared by the kernel).
// `stable_rows` >= 0 promises that the kernels enqueued on `stream` since the last full
// dependency are decode steps of this cache which write no row below `stable_rows`; the kernel
// may then read those rows while the earlier steps are still running.
int decode_step_impl(const void *q, const void *k_new, const void *v_new, ec_cache *c, float scale, void *out,
                     int *evicted_slot, int *slot_written, void *ws, size_t ws_bytes, void *stream, int stable_rows,
                     bool fresh_ws)
{
    if (!q || !k_new || !v_new || !c || !out || !evicted_slot) return EC_ERR_NULL;
    int cst = ec::check_cache(c);
    if (cst != EC_OK) return cst;
    const bool ratio = (c->policy == EC_POLICY_RATIO);
    if (!(scale > 0.f) || !isfinite(scale)) return EC_ERR_ARG;
    if (!aligned(q, 16) || !aligned(k_new, 16) || !aligned(v_new, 16) || !aligned(out, 16)) return EC_ERR_ALIGN;
    if (!ws || ws_bytes < ec_decode_workspace(c)) return EC_ERR_WORKSPACE;
    if (!aligned(ws, 256)) return EC_ERR_ALIGN;

    // Fixed-point elimination: queue position len - offset leaves, i.e. the oldest of the
    // `offset` newest rows. Older rows never move, so only the newest rows' slots are tracked:
    // a ring over [budget-offset, budget) for the fixed budget, an explicit ring of slots
    // when the cache may still grow.
    int slot, evicted;
    if (ratio) {
        // Algorithm 1: del_num = int(seq_len - n * retained_fraction), after the append
        const double del = (double)(c->len + 1) - (double)(c->n_tot + 1) * c->keep_ratio;
        if ((int)del >= 1) {
            slot = c->recent_slots_host[c->recent_head];
            evicted = slot;
        } else {
            if (c->len >= c->cap) return EC_ERR_ARG;     // no room left to grow
            slot = c->len;
            evicted = -1;
        }
    } else if (c->len < c->budget) {
        slot = c->len;
        evicted = -1;
    } else {
        slot = c->budget - c->offset + c->ring_head;
        evicted = slot;
    }
    const int units = c->N * c->H;
    const int splits = ec::decode_splits(units, c->len + 1);
    const size_t counter_bytes = round256((size_t)units * sizeof(int));
    int *counters = static_cast<int *>(ws);
    float *partials = reinterpret_cast<float *>(static_cast<char *>(ws) + counter_bytes);
    cudaError_t e;
    if (fresh_ws && ec::decode_splits(units, c->cap + 1) > 1) {
        e = cudaMemsetAsync(counters, 0, (size_t)units * sizeof(int), (cudaStream_t)stream);
        if (e != cudaSuccess) return EC_ERR_CUDA;
    }
    e = ec::launch_decode(q, k_new, v_new, c->Kc, c->Vc, units, c->D, c->cap, c->len, slot, stable_rows, scale, out,
                          partials, counters, splits, (cudaStream_t)stream);
    if (e != cudaSuccess) return EC_ERR_CUDA;
    if (ratio) {
        if (c->queue_slots_host) {
            // queue order: the row that leaves sits `offset` places before the end (it is the oldest of
            // the `offset` newest rows); the rows behind it move up, the new row joins at the tail
            int *order = c->queue_slots_host;
            if (evicted >= 0) {
                for (int j = c->len - c->offset; j < c->len - 1; ++j) order[j] = order[j + 1];
                order[c->len - 1] = slot;
            } else {
                order[c->len] = slot;
            }
        }
        // the new row is now the newest; the ring's oldest entry either left or stops being tracked
        c->recent_slots_host[c->recent_head] = slot;
        c->recent_head = (c->recent_head + 1) % c->offset;
        if (evicted < 0) c->len += 1;
        c->n_tot += 1;
    } else if (evicted >= 0) {
        c->ring_head = (c->ring_head + 1) % c->offset;
    } else {
        c->len += 1;
    }
    c->step += 1;
    *evicted_slot = evicted;
    if (slot_written) *slot_written = slot;
    return EC_OK;
}

}  // namespace

extern "C" {

int ec_decode_step(const void *q, const void *k_new, const void *v_new, ec_cache *c, float scale, void *out,
                   int *evicted_slot, int *slot_written, void *ws, size_t ws_bytes, void *stream)
{
    ec::NvtxRange nvtx_range("ec_decode_step");
    return decode_step_impl(q, k_new, v_new, c, scale, out, evicted_slot, slot_written, ws, ws_bytes, stream, -1, true);
}

int ec_decode_steps(const void *q, const void *k_new, const void *v_new, int steps, ec_cache *c, float scale,
                    void *out, int *evicted_slots, void *ws, size_t ws_bytes, void *stream)
{
    ec::NvtxRange nvtx_range("ec_decode_steps");
    if (steps < 0) return EC_ERR_ARG;
    int cst = ec::check_cache(c);
    if (cst != EC_OK) return cst;
    const size_t stride = (size_t)c->N * c->H * c->D * 2;   // bytes of one [N, H, D] bf16 step
    // Rows no step of this call will write: new rows go to the slots of the `offset` most recent
    // rows (the ring of a full fixed-budget cache, the tracked recent slots of the ratio policy) or
    // are appended at len and beyond. The first step knows nothing about the kernel before it.
    int stable = c->len;
    if (c->policy == EC_POLICY_RATIO) {
        if (c->recent_slots_host && c->offset >= 1)
            for (int i = 0; i < c->offset; ++i) stable = stable < c->recent_slots_host[i] ? stable : c->recent_slots_host[i];
    } else if (c->budget - c->offset < stable) {
        stable = c->budget - c->offset;
    }
    if (stable < 0) stable = 0;
    for (int s = 0; s < steps; ++s) {
        int ev = -1, slot = -1;
        int st = decode_step_impl(static_cast<const char *>(q) + s * stride, static_cast<const char *>(k_new) + s * stride,
                                  static_cast<const char *>(v_new) + s * stride, c, scale,
                                  static_cast<char *>(out) + s * stride, &ev, &slot, ws, ws_bytes, stream,
                                  s == 0 ? -1 : stable, s == 0);
        if (st != EC_OK) return st;
        if (evicted_slots) evicted_slots[s] = ev;
    }
    return EC_OK;
}

}  // extern "C"
