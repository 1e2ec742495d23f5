/*
 * spd.h -- C ABI of the partitioned decode-attention library (libspd.so) for NVIDIA B200 (sm_100a).
 *
 * The library computes one decode step of attention split across two KV partitions, as in
 * Secure Partitioned Decoding: every user's private ("input") partition holds the KV of its
 * prompt, the public ("output") partition holds the KV of generated tokens.  A partition yields a
 * partial result per (user, query head): an unnormalised output O, the running maximum m of the
 * scaled scores and the sum l of exp(score - m).  Two partials merge by log-sum-exp rescaling into
 * exactly the attention over the concatenated keys (Theorem 1, Eq. 1; stabilised form Sec. 4.2).
 *
 * Conventions for every call
 *   - "device" pointers are CUDA device memory owned by the caller, 16-byte aligned (pools 128-byte
 *     aligned).  The library allocates and frees no device memory.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t cast to void*, NULL = default stream)
 *     and return without waiting, except where stated.
 *   - Host-checkable mistakes (null pointer, unsupported shape, workspace too small) return an error
 *     code and launch nothing.  Mistakes only the device can see (a page index outside the pool, a
 *     length larger than the pages listed) never fault: the user concerned gets zeros as output, and
 *     a sticky flag is raised in the workspace, read by spd_query_device_status().
 *   - Layouts:  q [batch][num_q_heads][head_dim] in `dtype`;
 *               pools [num_pages][num_kv_heads][page_size][head_dim] in `dtype`;
 *               token t of user u lives in page page_indices[page_indptr[u] + t / page_size],
 *               slot t % page_size; slots at or beyond seq_lens[u] are never used in a result.
 *   - Query head h reads KV head h / (num_q_heads / num_kv_heads).
 *   - m and l are in natural-log units of the scaled score, so a partial can be handed from one
 *     call (or process) to another as is.  An empty partition gives O = 0, m = -inf, l = 0.
 *   - Supported: head_dim 64 or 128, page_size 16, dtype F32 or BF16 (q and KV alike),
 *     num_q_heads a multiple of num_kv_heads with a group size of 1, 2, 4, 8 or a multiple of 8.
 *   - Stream order.  The attention kernel is launched with programmatic stream serialisation: the part of it
 *     that only READS the lengths, the page tables and the KV pools may start while the previous kernel on the
 *     stream is still finishing; q, an incoming partial, the workspace and the outputs are touched only after
 *     that kernel has completed.  If a kernel of yours on the same stream writes lengths, page tables or KV rows
 *     immediately before a call, launch in plain stream order: spd_set_programmatic_launch(0), or SPD_NO_PDL=1
 *     in the environment.  Where the library's own calls write such inputs (the appends), they order themselves.
 *   - Threads.  Calls may come from several host threads, also from threads that have made no CUDA call of their
 *     own yet (the library makes the current device's context current on such a thread at its first call); calls
 *     that share a workspace must be ordered by the caller (one stream at a time per workspace).  Each workspace keeps a small table of streaming rates that
 *     sizes the next call's shares; it is rotated by a per-workspace launch count held on the host, so calls on
 *     other workspaces or streams never disturb it.
 *   - CUDA graphs.  Every call may be captured.  What is decided on the host at call time is then frozen into
 *     the graph: the call id (a user flagged in one replay stays flagged in later replays until the workspace's
 *     flags are cleared by spd_query_device_status), which third of the rate table a launch reads and writes
 *     (replays keep rotating correctly among the launches of one graph; shares keep following the rates that
 *     those launches leave), and the plan mode of the *_planned calls.
 */
#ifndef SPD_H_
#define SPD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SPD_OK = 0,
    SPD_ERR_INVALID_ARG = 1,   /* null pointer, negative size, misaligned pointer            */
    SPD_ERR_UNSUPPORTED = 2,   /* shape or dtype outside the supported set                     */
    SPD_ERR_WORKSPACE = 3,     /* workspace smaller than spd_workspace_size() reports          */
    SPD_ERR_BAD_PAGE = 4,      /* device saw a page index or length out of range (sticky flag) */
    SPD_ERR_CUDA = 5,          /* a CUDA runtime or driver call failed                         */
    SPD_ERR_TIMEOUT = 6,       /* a bounded wait inside a kernel ran out (sticky flag)         */
    SPD_ERR_PLAN = 7           /* a call told to reuse a stored plan found none that fits (sticky flag) */
} spd_status;

typedef enum { SPD_F32 = 0, SPD_BF16 = 1 } spd_dtype;

typedef struct {
    int32_t   batch;          /* users in the batch (one query token each) */
    int32_t   num_q_heads;
    int32_t   num_kv_heads;
    int32_t   head_dim;       /* 64 or 128 */
    int32_t   page_size;      /* 16 */
    spd_dtype dtype;          /* of q and of both pools */
    float     sm_scale;       /* multiplies q.k before the softmax (the paper's Eq. 1 has scale 1) */
} spd_shape;

/* One KV partition.  All pointers are device memory. */
typedef struct {
    const void    *k_pool;        /* [num_pages][num_kv_heads][page_size][head_dim] */
    const void    *v_pool;
    int32_t        num_pages;
    const int32_t *page_indptr;   /* [batch+1], page_indptr[0] = 0, non-decreasing                  */
    const int32_t *page_indices;  /* [page_indptr[batch]], each in [0, num_pages)                   */
    const int32_t *seq_lens;      /* [batch], 0 <= len <= page_size * (pages listed for the user)   */
} spd_paged_kv;

/* A partial attention result (device memory, fp32): the message between the two halves. */
typedef struct {
    float *o;   /* [batch][num_q_heads][head_dim], unnormalised */
    float *m;   /* [batch][num_q_heads] */
    float *l;   /* [batch][num_q_heads] */
} spd_partial;

/*
 * Bytes of device workspace the calls below need for `shape` on the current device.
 * The workspace holds the sticky status words, the table of streaming rates, the stored plans, per-user
 * flags, merge tickets, split-K scratch and the partial of a chained step; it does not depend on how many
 * tokens are cached.  Zero it once (cudaMemset) before first use, and again after an SPD_ERR_CUDA.  One
 * workspace serves one stream at a time.
 */
spd_status spd_workspace_size(const spd_shape *shape, size_t *bytes);

/*
 * Private partial attention (protocol step 3b; Fig. 3 step 4; Sec. 4.2): for every user and
 * query head, (O, m, l) over the user's private partition.  Long partitions are split across
 * warps and recombined by a second-level log-sum-exp merge.  `out` is fully overwritten; a user
 * flagged by the device gets the empty partial.  One kernel launch.
 */
spd_status spd_partial_attn(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                            spd_partial out, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Public partial attention batched over users, fused with the merge (protocol step 3c; Fig. 3
 * steps 3 and 5; Theorem 1): computes the partial over the public partition, merges it with `in`
 * (the private partial) and writes the normalised attention output
 *   out [batch][num_q_heads][head_dim] in `out_dtype` (F32 or BF16).
 * A user whose two partitions are both empty gets zeros.
 */
spd_status spd_service_attn_merge(const spd_shape *shape, const void *q, const spd_paged_kv *pub,
                                  spd_partial in, void *out, spd_dtype out_dtype,
                                  void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The merge on its own (Theorem 1, Eq. 1; maxima as in Sec. 4.2; Fig. 3 step 5), n-way: combines `n`
 * partials (1 <= n <= 8; `parts` is a HOST array of n structs holding device pointers) into the
 * normalised attention output.  For a caller that obtains the partials separately -- from other
 * processes, or from private and public halves run on different streams -- instead of letting
 * spd_service_attn_merge fuse the merge into the public half.  Rows whose partials are all empty give 0.
 * One small kernel on `cuda_stream`; no workspace.
 */
spd_status spd_merge_partials(const spd_shape *shape, int32_t n, const spd_partial *parts, void *out,
                              spd_dtype out_dtype, void *cuda_stream);

/*
 * One whole decode step of attention for one layer (protocol step 3, b and c): the private
 * partial, the public partial and their merge.  `fused` = 0 chains spd_partial_attn and
 * spd_service_attn_merge through a partial held in the workspace; `fused` != 0 streams both
 * partitions of a user through one running log-sum-exp (the same merge algebra applied tile by
 * tile), which saves the round trip of the partial.  Same result up to fp32 rounding order.
 */
spd_status spd_decode_step(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                           const spd_paged_kv *pub, void *out, spd_dtype out_dtype, int32_t fused,
                           void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The same three calls with the plan under the caller's control (the paper has no counterpart; the plan -- tiles
 * per user, their prefix sums, the share of the tile stream that each warp owns -- depends only on the two
 * seq_lens arrays, the shape and the GPU):
 *   SPD_PLAN_PER_CALL : derive the plan inside the kernel (what the plain calls do);
 *   SPD_PLAN_STORE    : derive it and leave it in the workspace;
 *   SPD_PLAN_REUSE    : load what the last SPD_PLAN_STORE call of the same kind (private only, public only, both
 *                       partitions) on this workspace and stream left, instead of deriving it.  The caller
 *                       states thereby that shape and every length are what they were at that call (page tables,
 *                       pools, q may differ).  A plan that was never stored, or was stored for another shape,
 *                       raises SPD_ERR_PLAN and the call writes nothing (a plain or PER_CALL call of the same
 *                       kind in between discards the stored plan); lengths that changed silently give
 *                       wrong results for the users concerned, possibly with SPD_ERR_PLAN or SPD_ERR_BAD_PAGE
 *                       raised (never a fault: every index is still checked).
 * Reuse pays for small calls, where deriving the plan is most of the time; large calls hide it anyway.
 */
typedef enum { SPD_PLAN_PER_CALL = 0, SPD_PLAN_STORE = 1, SPD_PLAN_REUSE = 2 } spd_plan_mode;
spd_status spd_partial_attn_planned(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                                    spd_partial out, spd_plan_mode plan, void *ws, size_t ws_bytes,
                                    void *cuda_stream);
spd_status spd_service_attn_merge_planned(const spd_shape *shape, const void *q, const spd_paged_kv *pub,
                                          spd_partial in, void *out, spd_dtype out_dtype, spd_plan_mode plan,
                                          void *ws, size_t ws_bytes, void *cuda_stream);
spd_status spd_decode_step_planned(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                                   const spd_paged_kv *pub, void *out, spd_dtype out_dtype, int32_t fused,
                                   spd_plan_mode plan, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Input-attention monitor (Sec. 2.4.4 and Sec. 7.1.1: watching how much attention the query pays to
 * the user's original instruction, inside the per-user process, to notice an instruction injected by
 * the service).  For every user, tokens [tok_lo[u], tok_hi[u]) of the PRIVATE partition are watched
 * (an empty or out-of-range interval watches nothing).  All pointers are device memory.
 *
 *   spd_partial_attn_watch : spd_partial_attn, plus out[u][h] = sum of exp(s_i - m) over the watched
 *                            tokens -- the watched part of l, in l's gauge; out / l is the share of the
 *                            private partition's softmax mass that sits on the watched tokens.
 *   spd_decode_step_watch  : spd_decode_step (fused), plus out[u][h] = share of the FULL softmax mass
 *                            (both partitions) that sits on the watched tokens, in [0, 1].
 * The attention output itself is what the unwatched calls give.
 */
typedef struct {
    const int32_t *tok_lo;   /* [batch] */
    const int32_t *tok_hi;   /* [batch] */
    float         *out;      /* [batch][num_q_heads] */
} spd_watch;
spd_status spd_partial_attn_watch(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                                  spd_partial out, const spd_watch *watch, void *ws, size_t ws_bytes,
                                  void *cuda_stream);
spd_status spd_decode_step_watch(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                                 const spd_paged_kv *pub, void *out, spd_dtype out_dtype,
                                 const spd_watch *watch, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The decision on top of the monitor (Sec. 2.4.4: an attack is detected whenever the monitored attention score
 * falls below an empirical threshold; the distraction effect shows in some specific heads).  HOST arrays only, no
 * device work: mass [batch][num_q_heads] is what a *_watch call produced, copied to the host by the caller;
 * head_mask [num_q_heads] (may be NULL = all heads) selects the heads that are watched; score[u] (may be NULL)
 * receives the mean of mass[u][h] over the selected heads and alarm[u] is set to 1 where that mean is below
 * `threshold`, else 0.  A user with no selected head, or a non-finite mean, raises the alarm.  Returns
 * SPD_ERR_INVALID_ARG for null mass or alarm, non-positive sizes or a threshold that is not a number.
 */
spd_status spd_watch_alarm(const float *mass, int32_t batch, int32_t num_q_heads, const uint8_t *head_mask,
                           float threshold, int32_t *alarm, float *score);

/*
 * Prefill (protocol step 2; Fig. 3 step 0): causal self-attention over every user's prompt, and the
 * hand-over of the prompt's K and V rows to the private paged cache that the decode calls read.
 *   q [total_tokens][num_q_heads][head_dim], k, v [total_tokens][num_kv_heads][head_dim]: the prompts of
 *   all users laid end to end; tok_indptr [batch+1] (device) gives each user's first token.
 *   out [total_tokens][num_q_heads][head_dim] in out_dtype: token i of a prompt attends to tokens 0..i of
 *   the same prompt (softmax of sm_scale * q.k, as in the decode calls).
 *   k_pool / v_pool / page tables: the private partition; token t of user u is stored in page
 *   page_indices[page_indptr[u] + t / page_size], slot t % page_size, and seq_lens[u] is set to the
 *   prompt's length.  A user whose listed pages cannot hold its prompt is skipped by the hand-over (its
 *   attention is still computed) and raises SPD_ERR_BAD_PAGE in the status words at the start of `ws`.
 *   tok_indptr must be non-decreasing and end at total_tokens; where it is not, the users before the first
 *   inconsistent one are served, the rows of that user and of all later ones are left unwritten, and the
 *   same status is raised.  Nothing is read or written out of bounds either way.
 * Supported: every shape the decode calls take, with sm_scale > 0 (else SPD_ERR_UNSUPPORTED).  Two kernels on
 * `cuda_stream`: the copy into the cache and the attention -- for BF16 with head_dim 128 on the tensor cores
 * (tcgen05 MMAs with accumulators in tensor memory), for FP32 prompts and for head_dim 64 on the FMA pipes (fp32
 * arithmetic throughout; a correctness path, not a fast one).
 */
spd_status spd_prefill_attn(const spd_shape *shape, int64_t total_tokens, const void *q, const void *k,
                            const void *v, const int32_t *tok_indptr, void *k_pool, void *v_pool,
                            int32_t num_pages, const int32_t *page_indptr, const int32_t *page_indices,
                            int32_t *seq_lens, void *out, spd_dtype out_dtype, void *ws, size_t ws_bytes,
                            void *cuda_stream);

/*
 * Append of the new token's K and V rows to a paged cache -- what the service does to its public
 * cache right before attention (protocol step 3a; Fig. 3 step 2), so that the new token attends to
 * itself through the public partition.  k_new, v_new: [batch][num_kv_heads][head_dim] in the shape's
 * dtype.  The row of user u lands at token position seq_lens[u] (page
 * page_indices[page_indptr[u] + seq_lens[u] / page_size], slot seq_lens[u] % page_size) and seq_lens[u]
 * grows by one, in place.  The caller provides the room: a user whose listed pages are already full
 * (or whose table is inconsistent) is left untouched and raises SPD_ERR_BAD_PAGE in the workspace's
 * status words.  One small kernel, enqueued on the stream in plain stream order (it starts after
 * every earlier call on that stream has finished with the cache).
 */
spd_status spd_append_kv(const spd_shape *shape, const void *k_new, const void *v_new, void *k_pool,
                         void *v_pool, int32_t num_pages, const int32_t *page_indptr,
                         const int32_t *page_indices, int32_t *seq_lens, void *ws, size_t ws_bytes,
                         void *cuda_stream);

/*
 * The append and the decode step in ONE launch (protocol steps 3a, 3b and 3c; Fig. 3 steps 2 to 5): the fused
 * spd_decode_step over a public partition that already counts the new token, whose K and V rows are taken from
 * k_new / v_new ([batch][num_kv_heads][head_dim], shape dtype) instead of the cache, and written to the cache on
 * the way.  On return of the kernel the row of user u sits at token position seq_lens[u] of `pub` (the value
 * before the call) and seq_lens[u] has grown by one, in place, as with spd_append_kv; `pub`'s pools and seq_lens
 * are written although the struct declares them const.  A user whose listed pages are full, or who is flagged
 * for any other reason during the call (inconsistent table, page index outside a pool), gets zeros as output, no
 * append and an unchanged length, and raises SPD_ERR_BAD_PAGE.  `plan` as in the *_planned calls; a plan is
 * cut for the lengths INCLUDING the new token, so SPD_PLAN_REUSE fits a cache with the same lengths as the one
 * the storing call saw before ITS append.  A call that derives its plan starts in plain stream order.
 */
spd_status spd_decode_step_append(const spd_shape *shape, const void *q, const void *k_new, const void *v_new,
                                  const spd_paged_kv *priv, const spd_paged_kv *pub, void *out,
                                  spd_dtype out_dtype, spd_plan_mode plan, void *ws, size_t ws_bytes,
                                  void *cuda_stream);

/*
 * The service's whole share of a decode step in one launch (protocol steps 3a and 3c; Fig. 3 steps 2, 3 and 5):
 * spd_service_attn_merge with the append of the new token's K and V rows at its head -- the public partition counts
 * the new token, whose rows come from k_new / v_new and are written to the cache on the way, the public partial is
 * merged with `in` (the private partial that a per-user process computed meanwhile, which never sees the public
 * cache) and the attention output is written.  Lengths, flags, `plan` and stream order as for
 * spd_decode_step_append.
 */
spd_status spd_service_attn_merge_append(const spd_shape *shape, const void *q, const void *k_new,
                                         const void *v_new, const spd_paged_kv *pub, spd_partial in, void *out,
                                         spd_dtype out_dtype, spd_plan_mode plan, void *ws, size_t ws_bytes,
                                         void *cuda_stream);

/*
 * One token step over `num_layers` layers (protocol step 3 for every layer of the model; Fig. 3 steps 2 to
 * 5): for each layer in order, the new token's K and V rows are appended to that layer's public cache and the
 * layer's decode step runs, both inside one launch (spd_decode_step_append).  `layers` is a HOST array;
 * every pointer inside it is a device pointer that the caller owns.  Each layer brings its own caches,
 * page tables and lengths (layers[i].pub's pools and seq_lens are written by the append; two layers must not
 * share a seq_lens array), its own q and its own output.  In a model q of layer i+1 depends on layer i's output
 * through the weights; those are not this library's, so all inputs are taken as given and the driver only fixes
 * the order and the launch structure: num_layers kernels on `cuda_stream`, nothing else, so that a caller can
 * capture the whole token step in one CUDA graph and replay it (what is frozen into a graph is listed under
 * "CUDA graphs" at the top of this file).  The workspace is shared by the layers.  same_lengths != 0 states
 * that every layer's private and public seq_lens hold the same values as layer 0's (as in a model, whose layers
 * all cache the same tokens): the plan is then derived once, by layer 0, and loaded by the other layers
 * (SPD_PLAN_STORE / SPD_PLAN_REUSE above).  Stops at the first host-side error; device-side mistakes are
 * reported through spd_query_device_status as for the single calls.
 */
typedef struct {
    const void *q;             /* [batch][num_q_heads][head_dim]                                  */
    const void *k_new, *v_new; /* [batch][num_kv_heads][head_dim]: this layer's new token         */
    spd_paged_kv priv;         /* this layer's private (prompt) cache                             */
    spd_paged_kv pub;          /* this layer's public cache; pools and seq_lens are written       */
    void *out;                 /* [batch][num_q_heads][head_dim] in out_dtype                     */
} spd_layer;
spd_status spd_token_step(const spd_shape *shape, int32_t num_layers, const spd_layer *layers,
                          spd_dtype out_dtype, int32_t same_lengths, void *ws, size_t ws_bytes,
                          void *cuda_stream);

/*
 * spd_decode_step (fused) for a caller whose per-step data lives in HOST memory (no counterpart in
 * the paper, whose two processes exchange these arrays through the host on every layer).
 *
 * Everything that changes from step to step -- q, both partitions' page_indptr / seq_lens /
 * page_indices -- sits in ONE host buffer (pinned memory makes the copy asynchronous) at the offsets
 * that spd_step_blob_layout() reports, so that a step costs one host-to-device copy, one kernel and
 * one device-to-host copy (status words and output, which sit side by side in the blob).  The host
 * blob must start out zeroed; the call leaves its status block zeroed again.  The KV pools stay resident on the
 * device: `priv_pools` and `pub_pools` carry k_pool, v_pool and num_pages only (their table pointers
 * are ignored).  `device_blob` is device memory of layout->total_bytes, 256-byte aligned.
 *
 * A batch whose q or output comes to megabytes is served in two parts inside the call, so that the second part's q
 * goes up and the first part's output comes down (on a copy stream that the library keeps per host thread) while the
 * other part's kernel runs; the result is the same, row for row.
 *
 * The call copies host_blob[0, in_bytes) to the device, runs the step, copies status and output back
 * (the output to host_blob + layout->out), waits for the stream and returns the device status of
 * this step (*first_bad_user: lowest flagged user or -1; may be NULL).  The workspace's own sticky
 * status is not involved.
 */
typedef struct {
    int64_t priv_pages_listed, pub_pages_listed;   /* entries of the two page_indices arrays */
    size_t  q;                                      /* [batch][num_q_heads][head_dim], shape dtype */
    size_t  priv_indptr, priv_lens, priv_indices;   /* int32 [batch+1], [batch], [priv_pages_listed] */
    size_t  pub_indptr, pub_lens, pub_indices;
    size_t  status;                                 /* 256 bytes the caller keeps ZERO on the host */
    size_t  in_bytes;                               /* the inputs (and the status block) occupy [0, in_bytes) */
    size_t  out;                                    /* [batch][num_q_heads][head_dim], out_dtype */
    size_t  total_bytes;
} spd_step_blob;
spd_status spd_step_blob_layout(const spd_shape *shape, int64_t priv_pages_listed, int64_t pub_pages_listed,
                                spd_dtype out_dtype, spd_step_blob *layout);
spd_status spd_decode_step_host(const spd_shape *shape, const spd_step_blob *layout, void *host_blob,
                                void *device_blob, const spd_paged_kv *priv_pools,
                                const spd_paged_kv *pub_pools, spd_dtype out_dtype,
                                int32_t *first_bad_user, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Waits for `cuda_stream`, then reads and clears the workspace's sticky status.  Returns SPD_OK,
 * SPD_ERR_BAD_PAGE, SPD_ERR_TIMEOUT or SPD_ERR_PLAN; *first_bad_user (may be NULL) receives the lowest user
 * index that was flagged, or -1.  After a status other than SPD_OK the per-user flags and the merge tickets of
 * the workspace are cleared too, so the next call starts clean.
 */
spd_status spd_query_device_status(void *ws, void *cuda_stream, int32_t *first_bad_user);

/* Number of kernels the library has launched in this process (for accounting in benchmarks). */
int64_t spd_kernel_launch_count(void);

/*
 * Timing aid (no counterpart in the paper): between spd_profile_begin() and spd_profile_end()
 * every library call (at most `max_calls` of them; a chained decode step counts as two) has its
 * kernel bracketed by CUDA events on the caller's stream.  spd_profile_end() waits for the last
 * recorded call and returns the number of calls recorded and their summed kernel time in
 * milliseconds.
 */
spd_status spd_profile_begin(int32_t max_calls);
spd_status spd_profile_end(int32_t *calls, double *kernel_ms);

/*
 * spd_decode_step (fused) for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is a packaging of the same kernels.)
 *
 * Some hosts of this library may not call cudaMalloc: code that runs while a CUDA graph is being
 * captured, plug-ins of a serving engine that owns the whole memory pool and hands none out, and
 * sandboxed per-user workers that are given buffers but no right to grow their footprint.  For them
 * the workspace lives inside the library, in one statically declared device array of
 * SPD_STATIC_WS_BYTES bytes that every GPU loading the library holds until the process exits.  The
 * caller passes only inputs and the output buffer.
 *
 *   - Limit: the shape must need no more than SPD_STATIC_WS_BYTES of workspace (what
 *     spd_workspace_size() reports); otherwise the call launches nothing, prints one line to stderr
 *     and returns SPD_ERR_WORKSPACE.  On a 148-SM B200 that admits roughly
 *     batch * num_q_heads <= 12000 at head_dim 128.
 *   - The first call on each device looks up the array's device address (with that device current).
 *     Make that first call outside any stream capture.
 *   - All calls share the one array, and it keeps what the previous call left, laid out for the
 *     previous call's shape.  The call itself clears what must start at zero (the sticky status, the
 *     per-user flags and the merge tickets), so neither a flag raised by an earlier call nor tickets
 *     that an earlier call left drawn (a call that timed out, or one of another shape whose scratch lay
 *     where this call's tickets lie) leak into this one.  Two calls that overlap on the GPU
 *     (different streams, or different host threads without ordering) race on the array: order them.
 *   - The call allocates and frees nothing, on the device or through any library.
 *   - wait_and_check = 0: returns once the work is enqueued.  Non-zero: waits for the stream and
 *     returns the device status as spd_query_device_status() would (*first_bad_user as there).
 */
#define SPD_STATIC_WS_BYTES (16u << 20)
spd_status spd_decode_step_static(const spd_shape *shape, const void *q, const spd_paged_kv *priv,
                                  const spd_paged_kv *pub, void *out, spd_dtype out_dtype,
                                  int32_t wait_and_check, int32_t *first_bad_user, void *cuda_stream);

/*
 * Measurement aid (no counterpart in the paper): which arithmetic the bf16 kernels use from now on,
 * process-wide.  0 (default) = tensor cores (mma.sync, fp32 accumulate); 1 = the FMA pipes with K and V
 * widened to fp32 on the fly.  Same tiles, same memory traffic, same results within tolerance; path 1
 * exists to show where the tensor cores are needed (it falls behind HBM as the GQA group grows).
 */
spd_status spd_set_bf16_math(int32_t path);

/*
 * Tuning and test aid (no counterpart in the paper): query rows per CTA of spd_prefill_attn from now on,
 * process-wide.  0 (default) = chosen per call from the mean prompt length (256 rows, two tiles sharing
 * their K/V loads, from 768 tokens on, else 128); 128 or 256 force one tensor-core kernel; 8 forces the FMA-pipe
 * kernel (the one FP32 and head_dim 64 always take) for BF16 with head_dim 128 too.  All compute the same thing
 * within tolerance.
 */
spd_status spd_set_prefill_rows(int32_t rows);

/*
 * Test and tuning aid (no counterpart in the paper): how the tile stream is cut into shares from now on,
 * process-wide.  min_tiles_per_share: fewest page tiles (16 tokens each) a share may hold; 0 restores the default
 * (4); 1 lets every page become a piece of its own when the batch is small enough; a value at or above the
 * batch's tile count leaves one share, hence no second-level merge at all.  uniform_shares = 1 gives every CTA the
 * same weight and ignores the measured streaming rates: the cut points then depend on the lengths alone, and a
 * call repeated on the same inputs gives bit-identical results.
 */
spd_status spd_set_split(int32_t min_tiles_per_share, int32_t uniform_shares);

/*
 * Process-wide switch for programmatic stream serialisation of the attention kernel (see "Stream order" at the
 * top): 1 = on (default unless SPD_NO_PDL is set in the environment), 0 = plain stream order.
 */
spd_status spd_set_programmatic_launch(int32_t on);

/*
 * Debugging aids (no counterpart in the paper).  Both wait for `cuda_stream`.
 *   spd_debug_read_plan : the plan of the last call of kind `which` (0 = private partition only, 1 = public only,
 *     2 = both) on this workspace that derived its plan: *tiles = page tiles in the stream, *shares = warps that own a
 *     share, bnd[w] = first tile of share w for w in [0, *shares] (bnd[*shares] = *tiles); at most bnd_capacity
 *     entries are written.  Any of the three outputs may be NULL.
 *   spd_debug_sm_moves  : the rate table is indexed by CTA while the rates belong to SMs; *launches counts the
 *     attention launches on this workspace that could compare, *moves the CTAs among them that ran on another SM
 *     than the same CTA index did one launch earlier.
 */
spd_status spd_debug_read_plan(void *ws, int32_t which, void *cuda_stream, int32_t *tiles, int32_t *shares,
                               int32_t *bnd, int32_t bnd_capacity);
spd_status spd_debug_sm_moves(void *ws, void *cuda_stream, int64_t *launches, int64_t *moves);

/* Static text for a status code. */
const char *spd_status_string(spd_status status);

#ifdef __cplusplus
}
#endif
#endif /* SPD_H_ */
