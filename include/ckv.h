/*
 * ckv.h -- C ABI of the CollectiveKV decode-stage library for NVIDIA B200 (sm_100a).
 *
 * The library keeps, on one GPU, the learnable global K/V pool and the compressed
 * per-user caches of the paper (Sec. 4.2), and attends users' queries over the K/V it
 * rebuilds on chip:
 *
 *     K_c[i] = P_k[I_k[i]],  V_c[i] = P_v[I_v[i]]                    (Eq. Kc, inference branch)
 *     K = concat(K_u, K_c),  V = concat(V_u, V_c),  d_a = d_u + d_g   (Eq. K; user part first)
 *     out = attention(q, K, V)                                        (Sec. 4.2, last sentence)
 *
 * Full-width K/V never exist in device memory except through the test-only
 * ckv_materialize.
 *
 * Conventions
 *   - A "group" is one (layer, head) pair; every group has its own pool pair and its own
 *     index pair.  n_groups = layers * heads.
 *   - Indices are 0-based int32 at this boundary (the paper counts from 1).
 *   - Pointers marked [host] must be host memory.  Pointers marked [any] may be device
 *     memory or host memory (pinned or pageable); the library detects which and stages
 *     host data through its own device buffers on `stream`.  With host *output* memory the
 *     call returns after the copy has been enqueued; synchronise the stream before reading.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls enqueue work on it and return; ckv_cache_put* additionally wait for their own
 *     index validation (one 4-byte read-back).
 *   - The library copies what it is given: inputs may be released once the stream has
 *     passed the call.  Outputs are caller-owned.
 *   - Errors are return codes.  Nothing aborts, traps or throws across the boundary.  After
 *     any error the context is unchanged and stays usable (CKV_ERR_CUDA excepted: the CUDA
 *     context may be lost).
 *   - A context belongs to one device and may be used by one host thread at a time.  All calls
 *     on a context must be ordered on the GPU: pass the same stream, or chain the streams with
 *     events.  The context's scratch buffers, its plan tables and the storage that evicted or
 *     replaced users give back are reused by later calls in stream order only.
 */
#ifndef CKV_H_
#define CKV_H_

#include <stdint.h>

#if defined(__GNUC__)
#define CKV_API __attribute__((visibility("default")))
#else
#define CKV_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ckv_ctx ckv_ctx;

typedef enum {
    CKV_OK = 0,
    CKV_ERR_INVALID_ARG = 1,  /* NULL pointer, negative size, bad enum, offsets not monotone   */
    CKV_ERR_SHAPE = 2,        /* d_shared + d_user != head_dim, or a size that contradicts the
                                 pool already loaded                                           */
    CKV_ERR_STATE = 3,        /* call needs a pool and none is loaded                          */
    CKV_ERR_INDEX_RANGE = 4,  /* some pool index outside [0, n_entries)                        */
    CKV_ERR_UNKNOWN_USER = 5, /* user id has no cache entry                                    */
    CKV_ERR_OOM = 6,          /* device or host allocation failed                              */
    CKV_ERR_CUDA = 7,         /* a CUDA call failed; see ckv_last_cuda_error                   */
    CKV_ERR_UNSUPPORTED = 8,  /* configuration outside what the kernels were built for         */
    CKV_ERR_TOO_LARGE = 9     /* request beyond a fixed capacity (ckv_attend_static only)      */
} ckv_status;

typedef enum { CKV_F32 = 0, CKV_BF16 = 1 } ckv_dtype;

typedef enum {
    CKV_SOFTMAX = 0,      /* p = softmax_i(scale * <q, K[i]>),  out = sum_i p_i V[i]            */
    CKV_SILU_OVER_L = 1   /* out = (1/L_u) sum_i silu(scale * <q, K[i]>) V[i]  (HSTU-style)     */
} ckv_mode;

typedef struct {
    int32_t n_groups;     /* >= 1                                                               */
    int32_t head_dim;     /* d_a = d_shared + d_user; one of 16, 32, 64, 128                    */
    int32_t dtype;        /* ckv_dtype of pool, user K/V and queries                            */
    int32_t out_dtype;    /* ckv_dtype of the outputs (fp32 accumulator, rounded once, RNE)     */
    int32_t mode;         /* ckv_mode                                                           */
    float scale;          /* multiplies <q, K[i]>; <= 0 selects the default:
                             1/sqrt(head_dim) for CKV_SOFTMAX, 1 for CKV_SILU_OVER_L            */
    int32_t device;       /* CUDA device ordinal                                                */
} ckv_config;

/* Create / destroy a context on cfg->device.  ckv_destroy(NULL) is a no-op.
 * Errors: INVALID_ARG, UNSUPPORTED (head_dim), CUDA, OOM. */
CKV_API ckv_status ckv_create(const ckv_config* cfg, ckv_ctx** out);
CKV_API ckv_status ckv_destroy(ckv_ctx* ctx);

/*
 * Global K/V pool P_k, P_v (Sec. 4.2: learnable tables shared by all users that stay in GPU
 * memory at inference).
 *   pool_K, pool_V [any] : [n_groups][n_entries][d_shared], contiguous, ctx dtype.
 * The pool is copied into the library's own row layout (full head_dim-wide rows whose first
 * d_user slots are zero).  To keep it resident in L2 the call raises this process's persisting-L2
 * carve-out on the device to the pool's size (cudaLimitPersistingL2CacheSize, capped by the device;
 * put back when the last context on the device is destroyed); see option "l2_persist".  Fixes
 * d_user = head_dim - d_shared and
 * the stored index width (16 bit when n_entries <= 65536, else 32 bit).  May be called again
 * with the same n_entries and d_shared to refresh the values; any other reload while users
 * are cached is CKV_ERR_SHAPE.
 * Errors: INVALID_ARG (NULL, n_entries < 1), SHAPE (d_shared outside [1, head_dim]), OOM, CUDA.
 */
CKV_API ckv_status ckv_pool_load(ckv_ctx* ctx, const void* pool_K, const void* pool_V,
                         int32_t n_entries, int32_t d_shared, void* stream);

/*
 * Sharing only the keys or only the values (ablation on sharing keys or values, Sec. 5.5: "CollectiveK"
 * shares the keys and keeps classical values, "CollectiveV" the reverse).  As ckv_pool_load, with a shared
 * width per side:
 *   d_shared_k, d_shared_v : 0 = that side is not shared: it has no pool (its pool pointer is ignored and may be
 *       NULL) and no indices, and the cache calls take its full head_dim-wide rows as the "user" array of that
 *       side (user_K or user_V : [L][n_groups][head_dim]; idx_K or idx_V is ignored and may be NULL).
 *       Otherwise 1..head_dim as for ckv_pool_load; when both are non-zero they must be equal.
 *   The d_user argument of the cache calls is head_dim - max(d_shared_k, d_shared_v), the user-specific width
 *   of the shared side(s) (head_dim if no side is shared, which is a classical KV cache).
 * The blob of ckv_cache_export / ckv_cache_import then has an empty index section for a side that is not shared
 * and head_dim elements per entry in that side's user section; ckv_cache_bytes counts what is stored.
 * Decode runs on the CUDA-core, the warp-level tensor-core and the tcgen05 kernels (option "kernel" 0 to 3; the
 * warp-level kernel's TMA loader and the pool-side factorisation are not available).
 * Errors: as ckv_pool_load; SHAPE also for unequal non-zero widths.
 */
CKV_API ckv_status ckv_pool_load_sides(ckv_ctx* ctx, const void* pool_K, const void* pool_V, int32_t n_entries,
                                       int32_t d_shared_k, int32_t d_shared_v, void* stream);

/*
 * Store one user's compressed cache (Sec. 4.2, prefill output: global K/V indices plus
 * user-specific K/V), replacing any earlier entry of `user` (whose storage is reused by later
 * puts, imports and appends).
 *   idx_K, idx_V   [any] : int32 [L][n_groups]  (may alias each other)
 *   user_K, user_V [any] : [L][n_groups][d_user], ctx dtype; may be NULL iff d_user == 0
 *   L >= 0 (a user with an empty history is legal and attends to a zero output).
 * Errors: STATE (no pool), SHAPE (d_user != head_dim - d_shared), INVALID_ARG,
 *         INDEX_RANGE (cache unchanged), OOM, CUDA.
 */
CKV_API ckv_status ckv_cache_put(ckv_ctx* ctx, int64_t user, int32_t L,
                         const int32_t* idx_K, const int32_t* idx_V,
                         const void* user_K, const void* user_V, int32_t d_user, void* stream);

/*
 * Bulk form: n users whose histories are concatenated along the position axis.
 *   users [host] : int64 [n], distinct;  hist_off [host] : int64 [n+1], non-decreasing,
 *   hist_off[0] = 0;  arrays as in ckv_cache_put with L = hist_off[n].
 * All-or-nothing: on any error no user of the batch is stored.
 */
CKV_API ckv_status ckv_cache_put_batch(ckv_ctx* ctx, int32_t n, const int64_t* users,
                               const int64_t* hist_off,
                               const int32_t* idx_K, const int32_t* idx_V,
                               const void* user_K, const void* user_V, int32_t d_user,
                               void* stream);

/* Forget one user / all users (the pool stays).  Unknown user: CKV_ERR_UNKNOWN_USER.  The user's
 * storage goes to a free list (neighbouring free runs merge) and is reused first-fit, so a cache that
 * is updated continuously stays bounded by its live users plus fragmentation. */
CKV_API ckv_status ckv_cache_evict(ckv_ctx* ctx, int64_t user);
CKV_API ckv_status ckv_cache_clear(ckv_ctx* ctx);

/*
 * Decode: rebuild each listed user's K/V (Eq. Kc, Eq. K) on chip and attend the user's
 * queries over it, in the context's mode.  Candidates are independent target-attention
 * queries (Sec. 2.1: Q in R^{1 x d} per target item); there is no mask.
 *   users   [host] : int64 [n]   (a user may appear more than once)
 *   q_off   [host] : int32 [n+1], non-decreasing, q_off[0] = 0; user k owns query rows
 *                    q_off[k] .. q_off[k+1]-1
 *   queries [any]  : [q_off[n]][n_groups][head_dim], ctx dtype
 *   out     [any]  : [q_off[n]][n_groups][head_dim], ctx out_dtype, caller-allocated
 * With host memory for both `queries` and `out` and a few MB or more of queries, the request list
 * is cut into four ranges of consecutive users (eight from about 100 MB of queries on) whose upload,
 * kernels and download run on streams
 * of the library's own, so that the three overlap (pinned host memory is what makes the copies
 * asynchronous); `stream` is ordered before the first and behind the last of them, and the
 * results are the same bits.
 * A user with an empty history produces zero rows.  Results do not depend on how the
 * library splits long histories across thread blocks beyond fp32 rounding.  With kernel
 * families 1 to 3 (see option "kernel") they are bitwise reproducible from call to call for the
 * same context settings; family 4, which the library picks by itself for one query per user over
 * histories that are long against the pool, sums its weight histogram with shared-memory atomics
 * and can differ in the last bits from run to run (set option "kernel" to 2 where that matters).
 * A kernel whose internal bounded wait runs out cannot be reported by this (asynchronous) call:
 * read ckv_last_stat("device_errors") after synchronising when that matters.
 * Errors: STATE, INVALID_ARG, UNKNOWN_USER, OOM (workspace), CUDA.
 */
CKV_API ckv_status ckv_attend(ckv_ctx* ctx, int32_t n, const int64_t* users, const int32_t* q_off,
                      const void* queries, void* out, void* stream);

/*
 * Decode with a visible length per query: self-attention over the cached sequence (Sec. 2.1: in self-attention
 * models the s queries are projected from the sequence itself).  The paper does not restate the mask; this call
 * takes, for every query row, the number of leading history positions it attends:
 *   vis [any] : int32 [q_off[n]], row r of user k attends positions 0 .. vis[r]-1 of that user's history
 *               (values are clamped to [0, L_k]; causal self-attention over the whole history is
 *               vis = 1, 2, ..., L_k for the user's L_k queries; vis = 0 gives a zero row).
 * CKV_SOFTMAX normalises over the attended positions; CKV_SILU_OVER_L sums over them and still divides by the
 * user's history length L_k.  Everything else as ckv_attend; every gathering kernel serves this call (option
 * "kernel" 0 to 3; not the pool-side factorisation).  The tcgen05 kernel skips what lies behind the largest limit
 * of each block of 128 queries of a user, so causal self-attention costs about half of full attention.
 * Errors: as ckv_attend; INVALID_ARG also for vis == NULL with queries present.
 */
CKV_API ckv_status ckv_attend_visible(ckv_ctx* ctx, int32_t n, const int64_t* users, const int32_t* q_off,
                                      const int32_t* vis, const void* queries, void* out, void* stream);

/*
 * Decode without any allocation.  (The paper has no counterpart: this is a deployment variant of
 * ckv_attend, not a different computation.)
 *
 * ckv_attend may call cudaMalloc/cudaFree and cudaMallocHost: it grows a workspace for the partial
 * results of the split-along-history reduction and keeps per-request tables in device and pinned
 * memory it allocates.  Some callers cannot tolerate that: a serving thread inside a
 * latency-critical section (cudaMalloc and cudaFree synchronise the device), a process whose GPU
 * memory was handed in full to another allocator.  For them this entry point computes what
 * ckv_attend computes, but keeps those tables and partial results in a fixed array that is part
 * of the library's device image:
 *   - CKV_STATIC_SCRATCH_BYTES (8 MiB) per GPU that loads the library, held until the
 *     process exits, shared by every context and every call on that GPU;
 *   - limits: n <= CKV_STATIC_MAX_USERS (256) users per call, at most 4096 history chunks, and
 *     partial results (chunks x queries of every split user x n_groups x (head_dim + 2) floats)
 *     that fit the rest of the array.  Anything larger returns CKV_ERR_TOO_LARGE and
 *     enqueues nothing.  ("split_len" controls the chunk count; 0 = automatic.)
 *   - queries and out must be device memory (staging host buffers would need an allocation);
 *     host pointers return CKV_ERR_INVALID_ARG.
 *   - kernels: only the CUDA-core family (1) and the warp-level tensor-core family (2) run here
 *     (option "kernel" 0, 1 or 2; 3 and 4 return CKV_ERR_UNSUPPORTED: the tcgen05 kernel wants a
 *     work list and the factorised path tables whose sizes follow the request).  For requests
 *     that ckv_attend would give to family 3 or 4 the results agree within the usual tolerance,
 *     not bit for bit.
 * It calls no cudaMalloc, cudaFree or other allocating routine, and copies nothing from the
 * caller's host memory asynchronously: the request tables travel as kernel arguments of a small
 * kernel that writes them into the array (ceil(n / 80) launches of one thread block), followed by
 * the attend kernel and, for split histories, the merge kernel.  The first call on a device
 * looks up the array's device address (once per device, with that device current), which is also
 * when the CUDA driver may load the part of the library's device image that holds the array (the
 * 8 MiB leave the device's free memory at that moment, not later); make that first call during
 * start-up and outside any stream capture.
 * The array keeps the previous call's contents.  Nothing in it needs clearing: every entry
 * a call reads it has written itself.  Because all calls on a GPU share the array, two
 * calls whose kernels may overlap on the GPU (different streams, or different host threads)
 * race on it: serialise them (one stream, or events between streams).
 * Other arguments, results and errors are those of ckv_attend.
 */
#define CKV_STATIC_SCRATCH_BYTES (8u << 20)
#define CKV_STATIC_MAX_USERS 256
CKV_API ckv_status ckv_attend_static(ckv_ctx* ctx, int32_t n, const int64_t* users,
                                     const int32_t* q_off, const void* queries, void* out,
                                     void* stream);

/*
 * TEST ONLY -- the single path that writes full-width K/V to device memory: Eq. (Kc) and
 * Eq. (K) for one user.  K_out, V_out [any] : [L][n_groups][head_dim], ctx dtype.  The result
 * is a pure copy of input bits.
 */
CKV_API ckv_status ckv_materialize(ckv_ctx* ctx, int64_t user, void* K_out, void* V_out, void* stream);

/*
 * Prefill router (Sec. 4.3): the global-pool entry each of n history positions selects,
 *     idx_out[i][g] = the lowest j that maximises  x_i . W[g][j] + bias[g][j]
 * (one router per group; the K and the V router are two calls).  The n x n_entries score matrix is
 * never written.  Needs no context.
 *   x        device, bf16 [n][d_in]             inputs of the positions (d_in in {32, 64, 128})
 *   W        device, bf16 [n_groups][n_entries][d_in]   router weights, an entry's weights contiguous
 *   bias     device, fp32 [n_groups][n_entries], or NULL for none
 *   idx_out  device, int32 [n][n_groups]        what ckv_cache_put takes as idx_K / idx_V
 *   variant  0 = default (tcgen05 kernel), 1 = warp-level tensor-core kernel, 2 = tcgen05 kernel
 * Products are exact, sums fp32; entries whose scores are equal in that arithmetic resolve to the
 * lowest index.  The tcgen05 kernel's waits are bounded; the call reads its error word back and
 * therefore synchronises `stream` (variant 1 is only stream-ordered).
 * Errors: INVALID_ARG (sizes, null or host pointers), UNSUPPORTED (d_in), OOM, CUDA (also: a wait
 * inside the kernel ran out; idx_out is not valid then).
 */
CKV_API ckv_status ckv_route(int32_t device, int32_t n, int32_t n_groups, int32_t d_in, int32_t n_entries,
                             const void* x, const void* W, const float* bias, int32_t* idx_out, int32_t variant,
                             void* stream);

/*
 * Prefill, user-specific part (Sec. 4.2): the low-dimensional keys (or values) of n positions,
 *     out[i][g][c] = x_i . W[g][c] + bias[g][c],      c < d_out
 * (one call with the K weights, one with the V weights).  Needs no context.
 *   x     device, bf16 [n][d_in]                    d_in a multiple of 8, at most 256
 *   W     device, bf16 [n_groups][d_out][d_in]      d_out at most 16
 *   bias  device, fp32 [n_groups][d_out], or NULL
 *   out   device, bf16 [n][n_groups][d_out]         what ckv_cache_put takes as user_K / user_V
 * fp32 sums, result rounded to nearest even.  Stream-ordered.
 * Errors: INVALID_ARG, UNSUPPORTED (shape), CUDA.
 */
CKV_API ckv_status ckv_project(int32_t device, int32_t n, int32_t n_groups, int32_t d_in, int32_t d_out,
                               const void* x, const void* W, const float* bias, void* out, void* stream);

/*
 * Appends L_new positions (new interactions) behind a cached user's history; arguments as for
 * ckv_cache_put, describing only the new positions.  The user's compressed cache moves to other
 * storage holding the old and the new positions; the old storage is reused by later calls.
 * Synchronises `stream`.
 * Errors: INVALID_ARG, STATE (no pool), SHAPE (d_user), UNKNOWN_USER, INDEX_RANGE (an index
 * outside [0, n_entries); the user keeps the old history), OOM, CUDA.
 */
CKV_API ckv_status ckv_cache_append(ckv_ctx* ctx, int64_t user, int32_t L_new, const int32_t* idx_K,
                                    const int32_t* idx_V, const void* user_K, const void* user_V, int32_t d_user,
                                    void* stream);

/*
 * Decode-stage load path (Sec. 4.4: T_load(s d_u + s) + T_index): a serving system keeps the
 * compressed caches in host memory and loads the users of a request batch before attending.
 * A blob is the packed form of n users' caches exactly as the library stores them, so loading it
 * is four plain copies and no packing kernel.  Layout, for the users in the order given, with
 * units(u) = n_groups * round_up(L_u, 32):
 *     [ K indices of all users | V indices | user-specific K | user-specific V ]
 * each section holding units(u) entries per user back to back, an entry being [group][position]
 * within a user (2- or 4-byte indices as stored, d_user elements for the user parts; padding
 * positions hold index 0 and zeros), each section starting at a multiple of 256 bytes.  A blob is only meaningful for a context with the same n_groups, head_dim, dtype and
 * pool shape (n_entries, d_shared) as the one that exported it.
 *
 * ckv_cache_blob_bytes: size of the blob for histories of lengths L[0..n) (host array).
 * ckv_cache_export: writes the blob of n cached users to `blob` (host or device memory, `bytes`
 *   must equal ckv_cache_blob_bytes of their lengths); stream-ordered, synchronise before reading.
 * ckv_cache_import: stores n users from `blob` (host -- pinned for an asynchronous copy -- or
 *   device memory) under the given ids, replacing users that exist.  The stored indices are
 *   range-checked on the device; the call returns after that check (it synchronises `stream`).
 * Errors: INVALID_ARG (null pointers, n < 0, negative length, wrong `bytes`), STATE (no pool),
 *   UNKNOWN_USER (export), INDEX_RANGE (import: an index >= n_entries; nothing is stored),
 *   OOM, CUDA.
 */
CKV_API ckv_status ckv_cache_blob_bytes(ckv_ctx* ctx, int32_t n, const int32_t* L, int64_t* bytes);
CKV_API ckv_status ckv_cache_export(ckv_ctx* ctx, int32_t n, const int64_t* users, void* blob, int64_t bytes,
                                    void* stream);
CKV_API ckv_status ckv_cache_import(ckv_ctx* ctx, int32_t n, const int64_t* users, const int32_t* L,
                                    const void* blob, int64_t bytes, void* stream);

/* History length of a cached user.  Errors: UNKNOWN_USER. */
CKV_API ckv_status ckv_user_length(ckv_ctx* ctx, int64_t user, int64_t* L);

/*
 * Storage accounting over all cached users (Sec. 5.1 compression rate, Sec. 4.4 load size):
 *   compressed = bytes of stored indices + user-specific K/V (padding excluded)
 *   full_width = bytes a classical cache would hold: 2 * positions * n_groups * head_dim * e
 */
CKV_API ckv_status ckv_cache_bytes(ckv_ctx* ctx, int64_t* compressed, int64_t* full_width);

/*
 * Tuning and test knobs (integers).  Unknown name: INVALID_ARG.
 *   "split_len"    positions per history chunk for the split-along-history reduction;
 *                  0 = choose automatically (default)
 *   "kernel"       0 = choose by queries per user (default); 1 = CUDA-core kernel;
 *                  2 = warp-level tensor-core kernel; 3 = tcgen05 kernel; 4 = pool-side
 *                  factorisation (one query per user: per-user score and weight tables over the
 *                  pool replace the row gathers; chosen by default when histories are long against
 *                  the pool; its weight histogram is summed with shared-memory atomics, so the last
 *                  bits can differ from run to run).  ckv_attend returns UNSUPPORTED if the forced
 *                  kernel cannot take the request.
 *   "mma_loader"   how the warp-level tensor-core kernel brings pool rows into shared memory:
 *                  0 or 1 = 16-byte asynchronous copies through L1 (default), 2 = TMA row gathers
 *                  (UNSUPPORTED from ckv_attend if the driver cannot encode the tensor maps);
 *                  the results are the same bits either way
 *   "l2_persist"   1 (default) = every ckv_attend puts an access-policy window over the pool
 *                  (persisting hits) on the caller's stream while it enqueues its kernels and restores
 *                  the stream's previous window before it returns; 0 = leave the stream alone
 *   "time_kernels" 1 = record CUDA events around the kernels of each ckv_attend (see ckv_last_stat)
 */
CKV_API ckv_status ckv_set_option(ckv_ctx* ctx, const char* name, int64_t value);
CKV_API ckv_status ckv_get_option(ckv_ctx* ctx, const char* name, int64_t* value);

/*
 * Introspection for tests and the benchmark.  Counters describe the most recent
 * ckv_attend: "launches" (kernels enqueued), "work_items", "split_items" (items that went
 * through the partial-result workspace), "kernel" (family that ran: 1 to 4), "mma_loader"
 * (loader the last warp-level tensor-core launch used: 1 or 2),
 * "workspace_bytes", "plan_cache_hit", "alloc_calls" (device or pinned-host allocations the call
 * made: 0 once its buffers have reached their size), "l2_window" (1 if the pool's L2 window was on
 * the stream for the call), "pipeline_ranges" (ranges of users a host-buffer call was cut into: 1, 4 or 8); "arena_capacity_units", "arena_used_units", "arena_free_runs" (state of
 * the compressed-cache storage, in (position, group) units); with option "time_kernels" also
 * "main_kernel_ns" and
 * "combine_kernel_ns" (device time of the attend kernel and of the split-merge kernel; the
 * query waits for that attend to finish; CKV_ERR_STATE if nothing was timed).
 * "device_errors" (not tied to the last call): non-zero once a kernel of this context gave up
 * on one of its internal bounded waits -- its outputs are then invalid; synchronises the device.
 * (Diagnostics of the tcgen05 kernel: bits 0-3 name the roles that gave up, bits 8-11 the wait
 * that ran out first.)
 * In the range-checked build of the library (build.py --bounds) bit 32 of it reports an index, row
 * or shared-memory offset that a kernel found outside its bound (the access is then redirected, not
 * performed).
 */
CKV_API ckv_status ckv_last_stat(ckv_ctx* ctx, const char* name, int64_t* value);

CKV_API const char* ckv_strerror(ckv_status s);
/* Text of the last CUDA error seen by this context ("" if none). */
CKV_API const char* ckv_last_cuda_error(ckv_ctx* ctx);
/* Library version as major*10000 + minor*100 + patch. */
CKV_API int32_t ckv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CKV_H_ */
