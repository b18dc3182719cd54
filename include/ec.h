/*
 * ec.h — C ABI of the Elastic Cache hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements the cache manager of "Efficient Inference of Vision
 * Instruction-Following Models with Elastic Cache" (arXiv 2407.18121), Sec. 3.3 and
 * Algorithm 1, as CUDA kernels:
 *
 *   ec_importance    per-head importance of every prompt key (Eq. 1 + column sums)
 *   ec_select_merge  anchor selection, bucket division (Eq. 2) and mean merge (Eq. 3)
 *                    into a dense compacted cache with an index map
 *   ec_decode_step   single-query attention over the compacted cache plus the new token,
 *                    followed by fixed-point elimination (in-place slot reuse)
 *
 * plus variants of each (importance on top of cached rows or from a known log-sum-exp,
 * shared populations and eviction-only compaction, a native multi-step decode loop, the
 * retention-ratio policy, host-resident tensors, a decode step with built-in scratch).
 *
 * Conventions shared by every call
 *  - Pointers named "dev" are CUDA device pointers of the current device; "host" pointers
 *    are ordinary host memory. The caller owns every buffer. No call allocates device
 *    memory, and no call depends on an earlier one except through the buffers and the
 *    ec_cache struct the caller passes (the library only caches a driver entry point and,
 *    for ec_decode_step_noalloc, the address of its built-in scratch).
 *  - bf16 tensors are passed as `const void*` to 2-byte elements, row-major, innermost
 *    dimension contiguous, base address 16-byte aligned. D (head_dim) is 64 or 128.
 *  - N counts independent problems (batch x layers folded), H heads per problem. A "unit"
 *    is one (problem, head) pair; units never interact except through EC_LAYER_SHARED.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream). Calls only enqueue
 *    work; they return after launch. Errors detectable on the host are returned at once and
 *    nothing is launched; in that case outputs are untouched.
 *  - Every function returns an ec_status as int. No function throws, aborts or prints.
 *  - Workspace: each call states its scratch need through the matching *_workspace query;
 *    the caller passes a device buffer of at least that many bytes, 256-byte aligned. The
 *    first 256 bytes of an importance workspace hold a device status word (see
 *    ec_device_status).
 */
#ifndef EC_H_
#define EC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    EC_OK = 0,
    EC_ERR_NULL = 1,      /* a required pointer is NULL                                  */
    EC_ERR_SHAPE = 2,     /* a dimension is out of the supported range                   */
    EC_ERR_ALIGN = 3,     /* a pointer is not 16-byte (workspace: 256-byte) aligned      */
    EC_ERR_ARG = 4,       /* a scalar argument is out of range                           */
    EC_ERR_WORKSPACE = 5, /* workspace missing or smaller than the query reports         */
    EC_ERR_CUDA = 6,      /* a CUDA runtime call failed (launch error, no device, ...)   */
    EC_ERR_TIMEOUT = 7,   /* a bounded device-side wait expired (see ec_device_status)   */
    EC_ERR_TOO_LARGE = 8  /* the problem does not fit the library's built-in scratch      */
} ec_status;

/* Static description of a status code; never NULL. */
const char *ec_status_string(int status);

/*
 * Number of anchors kept for a prompt of T tokens at retention ratio `keep_ratio`
 * (gamma of Sec. 3.3). Follows Algorithm 1's count of removed entries at the prompt call,
 * del = int(T - T*gamma), so the result is T - del, clamped to [1, T]. Host arithmetic in
 * double. Returns 0 when T < 1 or the ratio is not in [0, 1].
 */
int ec_keep_count(int T, double keep_ratio);

/* ---------------------------------------------------------------- importance ------- */

/* Bytes of device scratch ec_importance needs for these shapes (0 on invalid shapes). */
size_t ec_importance_workspace(int N, int H, int T, int D);

/*
 * Importance of every prompt key (Sec. 3.3, Eq. 1 and the definition that follows it):
 *   A[m][n] = exp(scale*<q_m,k_n>) / sum_{n'<=m} exp(scale*<q_m,k_n'>)   for n <= m, else 0
 *   scores[n] = sum_m A[m][n]
 * per unit. The T x T matrix is never stored: a first pass computes each query row's
 * log-sum-exp, a second pass accumulates the column sums.
 *
 *   Q_dev, K_dev   bf16 [N, H, T, D]                           (in)
 *   scores_dev     fp32 [N, H, T]                              (out)
 *   lse_dev        fp32 [N, H, T], natural log; may be NULL    (out, optional)
 *   scale          multiplies the dot product (the paper's Eq. 1 has none: pass 1.0 with
 *                  pre-scaled keys, or 1/sqrt(D) for a standard attention head)
 *   ws_dev         scratch of ec_importance_workspace bytes
 * Limits: 1 <= T <= 16384, N*H*T < 2^31, N*H < 2^24. Returns EC_OK or a host-detected error.
 */
int ec_importance(const void *Q_dev, const void *K_dev, float *scores_dev, float *lse_dev,
                  int N, int H, int T, int D, float scale,
                  void *ws_dev, size_t ws_bytes, void *stream);

/*
 * Importance when a new instruction of Tq tokens is encoded on top of P rows that are already
 * in the cache (Sec. 3.1: the instruction stage also takes in chat history; Eq. 1 with the
 * queries being the last Tq tokens): query m sees keys n <= m + P, and
 *   scores[n] = sum over the Tq queries of A[m][n],  n = 0 .. P+Tq-1.
 * The caller concatenates the cached rows and the new rows (K and, for ec_select_merge, V)
 * and compacts the P+Tq rows as usual. P = 0 is ec_importance.
 *   Q_dev       bf16 [N, H, Tq, D]                                   (in)
 *   K_dev       bf16 [N, H, P+Tq, D]                                 (in)
 *   scores_dev  fp32 [N, H, P+Tq]                                    (out)
 *   lse_dev     fp32 [N, H, Tq], natural log; may be NULL            (out, optional)
 *   ws_dev      scratch of ec_importance_workspace(N, H, Tq, D) bytes
 * Limits: Tq >= 1, P >= 0, P + Tq <= 16384.
 */
int ec_importance_prefix(const void *Q_dev, const void *K_dev, float *scores_dev, float *lse_dev,
                         int N, int H, int Tq, int P, int D, float scale,
                         void *ws_dev, size_t ws_bytes, void *stream);

/*
 * Other statistics of the attention a key receives (Sec. 3.2 "Importance Metrics" names
 * summation, moving average, maximum value and mean; the ablation on the importance metric
 * compares moving average, mean and sum). The paper gives no formulas; with A as in Eq. 1 and
 * the geometry of ec_importance_prefix (Tq queries, P + Tq keys, query m sees keys n <= m + P):
 *   EC_STAT_SUM             scores[n] = sum_m A[m][n]          (= ec_importance_prefix)
 *   EC_STAT_MEAN            the sum divided by the number of queries that can see key n,
 *                           Tq - max(0, n - P)
 *   EC_STAT_MAX             scores[n] = max_m A[m][n]
 *   EC_STAT_MOVING_AVERAGE  E <- beta*E + (1-beta)*A[m][.] over the queries in order, from
 *                           E = 0; scores = E after the last query, i.e. the sum with query m
 *                           weighted by (1-beta)*beta^(Tq-1-m). 0 < beta < 1; weights below
 *                           about 2^-125 count as zero
 * Arguments as ec_importance_prefix; `beta` is read for the moving average only. lse_dev, when
 * given, receives the plain log-sum-exp whatever the statistic. The statistic only changes
 * the scores: selection and merging take them as they take the sum.
 */
typedef enum { EC_STAT_SUM = 0, EC_STAT_MEAN = 1, EC_STAT_MAX = 2, EC_STAT_MOVING_AVERAGE = 3 } ec_statistic;

int ec_importance_statistic(const void *Q_dev, const void *K_dev, float *scores_dev, float *lse_dev,
                            int N, int H, int Tq, int P, int D, float scale, int statistic, double beta,
                            void *ws_dev, size_t ws_bytes, void *stream);

/*
 * The same importance when the caller already holds every query row's log-sum-exp, as a
 * prefill attention kernel produces it (the paper takes the attention probabilities from
 * the model's own forward pass, Algorithm 1 "Input"): only the column-sum pass runs, which
 * halves the contraction work.
 *   lse_dev   fp32 [N, H, T], natural log of sum_{n<=m} exp(scale*<q_m,k_n>), same `scale`  (in)
 * Other arguments, workspace size and limits as ec_importance.
 */
int ec_importance_from_lse(const void *Q_dev, const void *K_dev, const float *lse_dev, float *scores_dev,
                           int N, int H, int T, int D, float scale,
                           void *ws_dev, size_t ws_bytes, void *stream);

/*
 * The forward pass itself, for callers that want the library to produce it: causal attention of
 * the prompt tokens (Algorithm 1 "Input": the attention the method ranks tokens by is the one the
 * model's forward pass computes), with each row's log-sum-exp, and, when `scores_dev` is given,
 * the importance of Eq. 1 (Sec. 3.3) from that normaliser by the column-sum pass alone: three
 * contractions for attention + importance instead of four.
 *   out[m] = sum_{n <= m+P} softmax_n(scale*<q_m,k_n>) * v_n
 *   Q_dev       bf16 [N, H, Tq, D]                                                  (in)
 *   K_dev,V_dev bf16 [N, H, P+Tq, D]; P >= 0 earlier rows every query sees          (in)
 *   out_dev     bf16 [N, H, Tq, D]: fp32 accumulation, probabilities rounded to bf16
 *               before they meet V, one rounding of the normalised row at the end   (out)
 *   lse_dev     fp32 [N, H, Tq] natural log-sum-exp of every query row, nullable    (out)
 *   scores_dev  fp32 [N, H, P+Tq] importance as ec_importance_prefix gives it,
 *               nullable (no column-sum pass then)                                  (out)
 * Workspace, alignment, limits and status reporting as ec_importance_prefix
 * (ec_importance_workspace(N, H, Tq, D) bytes). Deterministic.
 */
int ec_prefill_attention(const void *Q_dev, const void *K_dev, const void *V_dev, void *out_dev, float *lse_dev,
                         float *scores_dev, int N, int H, int Tq, int P, int D, float scale,
                         void *ws_dev, size_t ws_bytes, void *stream);

/*
 * Synchronises `stream` and reports what the kernels recorded in the workspace's status
 * word: EC_OK, or EC_ERR_TIMEOUT if a bounded wait inside a kernel gave up (outputs are
 * then undefined but no out-of-bounds access happened). EC_ERR_CUDA on a runtime error.
 */
int ec_device_status(void *ws_dev, void *stream);

/*
 * Self-test of the failure path (no counterpart in the paper). The importance kernels wait
 * on hardware barriers with a time limit so that a lost signal can never hang the GPU. This
 * call enqueues a one-CTA kernel that waits, with that same routine, on a barrier nothing
 * completes; after `limit_us` microseconds (1 .. 1 000 000) the wait gives up, sets the status
 * word of `ws_dev` (any 256-byte-aligned device buffer of >= 256 bytes) and the kernel ends
 * normally. ec_device_status(ws_dev) then reports EC_ERR_TIMEOUT; the context stays usable.
 */
int ec_selftest_wait_timeout(void *ws_dev, unsigned limit_us, void *stream);

/* ---------------------------------------------------------------- select + merge ---- */

typedef enum {
    EC_PER_HEAD = 0,     /* every head ranks its own scores                              */
    EC_LAYER_SHARED = 1  /* scores are averaged over the heads of a problem first (the
                            paper's layer-wise population); all heads share the anchors  */
} ec_population;

size_t ec_select_merge_workspace(int N, int H, int T, int D, int n_keep, int population);

/*
 * Anchor selection, bucket division and merging (Sec. 3.3; Eq. 2; Eq. 3).
 *  1. anchors = the n_keep positions with the largest score (equal scores: the lower
 *     position wins), listed ascending. With protect_ends != 0, position 0 and (when
 *     n_keep >= 2) position T-1 are always anchors (Sec. 4.1, implementation details).
 *  2. bucket k = positions floor((t_{k-1}+t_k)/2)+1 .. floor((t_k+t_{k+1})/2), the first
 *     bucket starting at 0 and the last ending at T-1.
 *  3. row k of the compacted cache = arithmetic mean of the bucket's rows (fp32
 *     accumulation in position order, scaled by 1/size, one rounding to bf16), for K and for V.
 *
 *   K_dev, V_dev    bf16 [N, H, T, D]                                     (in)
 *   scores_dev      fp32 [N, H, T]                                        (in)
 *   n_keep          1..T (see ec_keep_count)
 *   Kc_dev, Vc_dev  bf16 [N, H, cap, D], rows 0..n_keep-1 written         (out), cap >= n_keep
 *   anchor_pos_dev  int32 [N, H, n_keep], ascending prompt positions      (out) = index map
 *   bucket_len_dev  int32 [N, H, n_keep], bucket sizes; may be NULL       (out, optional)
 * The inputs must not overlap the outputs.
 */
int ec_select_merge(const void *K_dev, const void *V_dev, const float *scores_dev,
                    int N, int H, int T, int D, int n_keep, int population, int protect_ends,
                    void *Kc_dev, void *Vc_dev, int cap,
                    int32_t *anchor_pos_dev, int32_t *bucket_len_dev,
                    void *ws_dev, size_t ws_bytes, void *stream);

/*
 * The general form of ec_select_merge, covering the variants of the paper's ablations
 * (Sec. 4.3: importance population; cache eviction versus cache merging):
 *   share       how many consecutive units rank one common score vector (the mean of their
 *               scores): 1 = head-wise, H = layer-wise, layers*H = one selection per sequence
 *               ("identical" for all layers; problems n = b*layers + l must be layer-minor).
 *               N*H must be a multiple of share.
 *   compaction  EC_COMPACT_MERGE: bucket means (Eq. 3).  EC_COMPACT_EVICT: the kept rows are
 *               the anchors' own rows and all other rows are dropped.
 * Everything else as ec_select_merge, which is this call with share = 1 or H and
 * EC_COMPACT_MERGE. Workspace: ec_select_compact_workspace.
 */
typedef enum { EC_COMPACT_MERGE = 0, EC_COMPACT_EVICT = 1 } ec_compaction;

size_t ec_select_compact_workspace(int N, int H, int T, int D, int n_keep, int share);

int ec_select_compact(const void *K_dev, const void *V_dev, const float *scores_dev,
                      int N, int H, int T, int D, int n_keep, int share, int protect_ends, int compaction,
                      void *Kc_dev, void *Vc_dev, int cap,
                      int32_t *anchor_pos_dev, int32_t *bucket_len_dev,
                      void *ws_dev, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------- decode ------------ */

/*
 * Host-side description of a compacted cache. Plain data: copy it to checkpoint it.
 * Rows live in device buffers Kc, Vc of shape bf16 [N, H, cap, D]; `len` rows are valid.
 * Because attention does not depend on row order, eviction does not shift rows: the new
 * row is written into the physical slot of the evicted one. Slots [budget-offset, budget)
 * form a ring that holds the `offset` most recent rows once the cache is full.
 */
typedef struct {
    void *Kc, *Vc;      /* device, bf16 [N, H, cap, D]                                   */
    int N, H, D, cap;
    int len;            /* valid rows per unit (same for all units)                      */
    int budget;         /* fixed-budget policy: rows kept after every step               */
    int offset;         /* rows that stay behind the truncation location (>= 1)          */
    int ring_head;      /* next ring slot to be reused, 0..offset-1                      */
    int64_t step;       /* decode steps taken                                            */
    /* retention-ratio policy only (see ec_cache_init_ratio); zero / NULL otherwise      */
    int policy;         /* EC_POLICY_FIXED or EC_POLICY_RATIO                            */
    int recent_head;    /* position of the oldest entry in recent_slots_host             */
    double keep_ratio;  /* retained fraction of all tokens seen                          */
    int64_t n_tot;      /* tokens seen so far, prompt included                           */
    int *recent_slots_host; /* caller-owned host array of `offset` ints: physical slots
                               of the `offset` newest rows, kept as a ring               */
    int *queue_slots_host;  /* optional (see ec_cache_track_order): caller-owned host array
                               of `cap` ints, the physical slot of every row in queue order */
} ec_cache;

typedef enum {
    EC_POLICY_FIXED = 0, /* the cache stays at `budget` rows: one row leaves every step  */
    EC_POLICY_RATIO = 1  /* the budget follows keep_ratio * tokens seen (Sec. 3.3: the
                            ratio is compared with a threshold after every new token)    */
} ec_policy;

/* Fills *c after validating: 2 <= budget <= cap, 0 <= len <= budget, 1 <= offset <= budget-1. */
int ec_cache_init(ec_cache *c, void *Kc_dev, void *Vc_dev, int N, int H, int D, int cap,
                  int len, int budget, int offset);

/*
 * Retention-ratio policy (Sec. 3.3 "Output Generation"; Algorithm 1: del_num =
 * int(seq_len - n * retained_fraction), evaluated after the new row was appended). A step
 * removes the row at the fixed truncation location only when del_num >= 1; otherwise the
 * cache grows by one row (up to cap; a step that would exceed cap returns EC_ERR_ARG).
 *   len                rows valid now (e.g. n_keep after ec_select_merge), len >= offset
 *   n_tot              tokens seen so far (the prompt length after the prompt call)
 *   recent_slots_host  host array of `offset` ints owned by the caller; it must stay valid
 *                      as long as *c is used. Rows that are no longer among the `offset`
 *                      newest never move again, so only these slots have to be tracked.
 */
int ec_cache_init_ratio(ec_cache *c, void *Kc_dev, void *Vc_dev, int N, int H, int D, int cap,
                        int len, int offset, double keep_ratio, int64_t n_tot, int *recent_slots_host);

/* Bytes of device scratch the decode calls need for this cache; depends on N, H, D and cap only.
 * 0 when those fields are out of range (N, H, cap >= 1; D 64 or 128; N*H < 2^24) or c is NULL. */
size_t ec_decode_workspace(const ec_cache *c);

/*
 * Makes a retention-ratio cache remember its queue order, so that a further instruction can be
 * encoded on top of it (ec_cache_concat). Under that policy a new row is appended while the cache
 * may grow and otherwise takes the slot of the row that leaves, so physical order and queue order
 * drift apart in a way only the sequence of grow / evict decisions determines; every decode step
 * then updates the list (an O(offset) shift on the host).
 *   c                  EC_POLICY_RATIO cache on which no step has been taken yet (c->step == 0):
 *                      its rows are still in slot order
 *   queue_slots_host   host array of c->cap ints owned by the caller, valid as long as *c is used;
 *                      entries 0 .. len-1 are filled here with 0 .. len-1
 * Returns EC_ERR_ARG for a fixed-budget cache (its order is implied by budget, offset and
 * ring_head) or when steps were already taken.
 */
int ec_cache_track_order(ec_cache *c, int *queue_slots_host);

/*
 * One generation step (Sec. 3.3 "Output Generation"; Algorithm 1, last branch):
 *   out = softmax(scale * q [Kc; k_new]^T) [Vc; v_new]      over len + 1 rows, per unit
 * then the new row joins the cache. If the cache was already at its budget, the row that
 * has exactly `offset` rows behind it (counting the new one) leaves: queue position
 * len - offset, which is the paper's fixed truncation location. Physically the new row
 * overwrites that row's slot; below budget it is appended at slot `len`.
 *
 *   q_dev, k_new_dev, v_new_dev  bf16 [N, H, D]                 (in)
 *   out_dev                      bf16 [N, H, D]                 (out)
 *   evicted_slot_host            physical slot that was overwritten, or -1 when the cache
 *                                was below budget (host int, written before return)
 *   slot_written_host            physical slot now holding the new row (may be NULL)
 * Updates c->len, c->ring_head, c->step on success. The struct is the caller's: every call
 * re-checks it (shape, alignment, policy fields) and returns an error instead of using a bad one.
 */
int ec_decode_step(const void *q_dev, const void *k_new_dev, const void *v_new_dev,
                   ec_cache *c, float scale, void *out_dev,
                   int *evicted_slot_host, int *slot_written_host,
                   void *ws_dev, size_t ws_bytes, void *stream);

/*
 * `steps` consecutive ec_decode_step calls issued from native code. Step s reads
 * q/k_new/v_new at element offset s*N*H*D of the three [steps, N, H, D] arrays and writes
 * out at the same offset. evicted_slots_host (may be NULL) receives `steps` ints.
 * All inputs of all steps must be complete on `stream` before the call: from the second step
 * on, a step starts reading its q/k_new/v_new and the cache rows that no step of the call
 * writes (everything but the slots of the `offset` most recent rows and the rows appended
 * during the call) while earlier steps of the call are still running; only those few rows, and
 * every write, wait for the step before.
 * The cache struct and the scalar arguments are checked before the first launch. A failure after
 * that (a CUDA launch error; under the retention-ratio policy a cache with no room left to grow)
 * ends the call at that step: the steps before it stay enqueued and c->step counts them.
 */
int ec_decode_steps(const void *q_dev, const void *k_new_dev, const void *v_new_dev, int steps,
                    ec_cache *c, float scale, void *out_dev, int *evicted_slots_host,
                    void *ws_dev, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------- host-resident tensors */

/*
 * The prompt call for tensors that start in host memory (Algorithm 1's prompt branch end to
 * end): copies Q, K, V to the caller's device staging buffers, then ec_importance and
 * ec_select_merge, then (optionally) copies the index map back. Everything is enqueued on
 * `stream`; pinned host memory makes the copies asynchronous.
 *   Q_host, K_host, V_host   host bf16 [N, H, T, D]                        (in)
 *   Q_dev, K_dev, V_dev      device staging of the same size                (scratch)
 *   anchor_pos_host          host int32 [N, H, n_keep]; may be NULL         (out, optional)
 *   ws_imp / ws_sel          workspaces of ec_importance / ec_select_merge
 * Other arguments as in those two calls.
 */
int ec_compress_host(const void *Q_host, const void *K_host, const void *V_host,
                     void *Q_dev, void *K_dev, void *V_dev, float *scores_dev,
                     int N, int H, int T, int D, float scale, int n_keep, int population, int protect_ends,
                     void *Kc_dev, void *Vc_dev, int cap, int32_t *anchor_pos_dev, int32_t *anchor_pos_host,
                     void *ws_imp_dev, size_t ws_imp_bytes, void *ws_sel_dev, size_t ws_sel_bytes, void *stream);

/*
 * ec_decode_steps for inputs and outputs in host memory. The steps are cut into chunks of
 * `chunk` steps (at most 31 chunks per call): the upload of later chunks (on upload_stream)
 * and the download of finished chunks (on download_stream) overlap the decoding of the
 * current chunk on `stream`. `stream` waits for the last download before the call's work
 * counts as complete on it.
 *   q_host, k_host, v_host, out_host   host bf16 [steps, N, H, D] (pinned for overlap)
 *   q_dev, k_dev, v_dev, out_dev       device staging of the same size
 *   upload_stream, download_stream     two further cudaStream_t, distinct from `stream`
 * The events the call creates are destroyed before it returns. Arguments are checked before the
 * first copy is enqueued (ec_compress_host likewise); on a later failure c->step tells how many
 * steps were enqueued.
 */
int ec_decode_steps_host(const void *q_host, const void *k_host, const void *v_host, void *out_host,
                         void *q_dev, void *k_dev, void *v_dev, void *out_dev, int steps, int chunk,
                         ec_cache *c, float scale, void *ws_dev, size_t ws_bytes,
                         void *stream, void *upload_stream, void *download_stream);

/* ---------------------------------------------------------------- history for a new instruction */

/*
 * The key/value history a further instruction is encoded against (Sec. 3.1: the instruction
 * stage takes in the chat history): the cache's rows in queue order, oldest first, followed
 * by the Tq rows of the new tokens. The result feeds ec_importance_prefix (P = c->len) and
 * ec_select_merge / ec_select_compact over T = c->len + Tq rows.
 *   c                      fixed-budget cache, or a retention-ratio cache that tracks its queue
 *                          order (ec_cache_track_order; without it EC_ERR_ARG); read only,
 *                          c->len >= 1
 *   K_new_dev, V_new_dev   device bf16 [N, H, Tq, D], 16-byte aligned, Tq >= 1
 *   K_all_dev, V_all_dev   device bf16 [N, H, c->len + Tq, D], written; must not overlap
 *                          the cache or the new rows
 * Row j < len of a unit comes from physical slot j while j < budget - offset or the cache is
 * not yet full, else from the ring: slot (budget - offset) + (ring_head + j - (budget - offset))
 * mod offset; for a retention-ratio cache from slot queue_slots_host[j] (the list is passed to
 * the copy kernels by value, a few hundred rows per launch, so the host array may change as soon
 * as the call returns). Rows are copied bit for bit. Asynchronous on `stream`.
 */
int ec_cache_concat(const ec_cache *c, const void *K_new_dev, const void *V_new_dev, int Tq,
                    void *K_all_dev, void *V_all_dev, void *stream);

/* ---------------------------------------------------------------- measurement aids */

/*
 * (No counterpart in the paper.) Reads `bytes` of device memory once with 16-byte streaming loads
 * and folds them into *sink_dev with XOR, so that timing the call gives the read-only bandwidth
 * this GPU sustains: the ceiling for the decode and merge kernels, which read far more than
 * they write (a copy, half reads and half writes, runs below it).
 *   buf_dev    device, 16-byte aligned, `bytes` long (bytes >= 16, a multiple of 16)
 *   sink_dev   device uint32, read-modify-written
 */
int ec_probe_read_stream(const void *buf_dev, size_t bytes, unsigned *sink_dev, void *stream);

/*
 * (No counterpart in the paper.) The same stream with writes mixed in: of every `write_every`
 * consecutive 256-byte rows read, one is also written to dst_dev, packed densely, which is the
 * read/write mix of the merge kernel at keep ratio 1/write_every (write_every = 0: no writes).
 * Timing it gives the ceiling for that mix on this GPU.
 *   dst_dev   device, 16-byte aligned, at least ceil(bytes/256 / write_every) * 256 bytes
 */
int ec_probe_mixed_stream(const void *buf_dev, size_t bytes, void *dst_dev, int write_every, unsigned *sink_dev,
                          void *stream);

/*
 * How many CTAs would share one unit's rows if ec_decode_step were called on *c now (1: one
 * CTA per unit, the layout of large batches; > 1: the split path with in-kernel merge).
 * 0 when *c is invalid.
 */
int ec_decode_splits(const ec_cache *c);

/* ---------------------------------------------------------------- no-allocation decode */

/*
 * (No counterpart in the paper: this is a deployment convenience.)
 *
 * ec_decode_step for callers that cannot allocate device memory and therefore cannot
 * provide the workspace: a server whose memory pool took the whole GPU at start-up, a
 * plug-in whose execute hook must not call cudaMalloc, a latency-critical loop that cannot
 * take cudaMalloc's device-wide synchronisation. Arguments, results and state updates are
 * those of ec_decode_step without ws/ws_bytes; the scratch is a fixed array inside the
 * library of ec_decode_noalloc_capacity() bytes (2 MiB, resident on every GPU that loads
 * the library until the process exits). The call itself allocates and frees nothing.
 *
 *  - Limit: ec_decode_workspace(c) must not exceed the capacity (at D = 128 about 4000
 *    units, N*H); otherwise EC_ERR_TOO_LARGE is returned and nothing is launched.
 *  - The first call on each device looks up the array's device address (a one-time runtime
 *    query, made with that device current). Make that first call outside any stream capture.
 *  - All calls on a device share the one array, which keeps whatever the previous call left
 *    there. Every call clears the per-unit arrival counters at the head of the array before
 *    its kernel (a memset node on `stream`, not an allocation) and rewrites the partial
 *    results it reads, so the caller clears nothing; but two calls whose kernels may run at
 *    the same time (different streams, different caches) race on the array: serialise them.
 */
size_t ec_decode_noalloc_capacity(void);
int ec_decode_step_noalloc(const void *q_dev, const void *k_new_dev, const void *v_new_dev,
                           ec_cache *c, float scale, void *out_dev,
                           int *evicted_slot_host, int *slot_written_host, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* EC_H_ */
