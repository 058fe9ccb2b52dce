/*
 * kvs.h -- C ABI of the shared-KV decode-attention library for NVIDIA B200 (sm_100a).
 *
 * The library implements the inference side of KVSharer (layer-wise KV cache
 * sharing): a per-model strategy says which layers' KV caches are replaced by
 * which earlier layers' caches (Section 3, Section 3.2, Fig. 3 of the paper).
 * During generation every layer still computes its own queries and runs the
 * unchanged attention, but a layer whose cache is replaced reads the keys and
 * values of its source layer and computes (appends) none of its own.
 *
 * Instead of copying a cache from layer to layer, the library keeps ONE cache
 * slot per layer that computes its own K/V and gives every layer an index into
 * those slots.  Results are those of the literal copy; memory is
 * (layers - shared layers) / layers of the unshared pool.
 *
 * Conventions for every call
 *   - returns a kvs_status; never throws, never aborts; on an error nothing
 *     has been written and no kernel has been launched;
 *   - "host" / "device" on a pointer says which memory it must point to;
 *   - the caller owns every buffer it passes (pool, workspace, q, k, v, out);
 *     the library owns only the kvs_ctx and small host tables;
 *   - work is enqueued on the given CUDA stream (a cudaStream_t passed as
 *     void*, NULL = the legacy default stream) and returns without waiting,
 *     except where a call says otherwise;
 *   - the calls of one context form ONE ordered chain on the GPU: issue them all on one stream, or,
 *     when the stream changes from one call to the next, make the new stream wait (event) for
 *     everything the previous call enqueued.  The library's kernels start early behind one another
 *     (see KVS_OPT_EARLY_START) and decide on the host which cached rows are already stable; that
 *     bookkeeping, and the shared workspace, assume this chain.  kvs_decode_attention_static is the
 *     one call that may run beside the chain (see there);
 *   - device pointers to q, k and v must be 16-byte aligned (INVALID_ARG otherwise): they are read
 *     with 16-byte vector loads and bulk copies;
 *   - all sequences of a batch are appended to together and have the same length, until
 *     kvs_evict makes the (sequence, head) units of a slot differ.
 *
 * Memory layout of the pool (device, caller-owned, bound with kvs_bind_memory):
 *   plane(slot, kv) with kv = 0 for K and 1 for V, each plane being
 *   [max_batch][n_kv_heads][row_stride][head_dim] elements of the storage
 *   type, row_stride = max_seq rounded up to a multiple of 128 rows;
 *   plane(slot, kv) starts (2 * slot + kv) * plane_bytes into the pool.
 *   One token row of one head is head_dim contiguous elements; the rows of one
 *   (sequence, head) are contiguous, so a tile of consecutive tokens is one
 *   contiguous run of bytes.
 */
#ifndef KVS_H_
#define KVS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct kvs_ctx kvs_ctx;

typedef enum {
    KVS_OK = 0,
    KVS_ERR_INVALID_ARG = 1,   /* NULL pointer, index or size out of range, unsupported shape */
    KVS_ERR_BAD_SHARE_MAP = 2, /* a source later than its target, or a negative entry        */
    KVS_ERR_STATE = 3,         /* call made in the wrong state (see each call)                */
    KVS_ERR_CAPACITY = 4,      /* an append would exceed max_seq                              */
    KVS_ERR_OOM = 5,           /* a bound buffer is smaller than kvs_required_bytes said      */
    KVS_ERR_CUDA = 6,          /* a CUDA runtime or driver call failed                        */
    KVS_ERR_TIMEOUT = 7,       /* a bounded device-side wait ran out (see kvs_last_device_status) */
    KVS_ERR_SCRATCH_LIMIT = 8, /* kvs_decode_attention_static: the call needs more than the built-in scratch */
    KVS_ERR_BOUNDS = 9         /* device status word only, bounds-checking build (-DKVS_DEBUG_BOUNDS) only: a
                                  kernel computed an offset outside the buffer it belongs to; the access was
                                  redirected or dropped and the launch ran on                               */
} kvs_status;

typedef enum { KVS_BF16 = 0, KVS_F32 = 1 } kvs_dtype;

typedef struct {
    int32_t n_layers;     /* L >= 1                                                 */
    int32_t n_q_heads;    /* Hq; a multiple of n_kv_heads; Hq/Hkv in 1..8 (3,5,6,7: bf16 only) */
    int32_t n_kv_heads;   /* Hkv >= 1                                               */
    int32_t head_dim;     /* 64 or 128                                              */
    int32_t max_batch;    /* largest batch any call will pass                       */
    int32_t max_seq;      /* capacity in tokens of every slot                       */
    int32_t dtype;        /* kvs_dtype: storage type of Q, K and V                  */
    float softmax_scale;  /* 0 means 1/sqrt(head_dim)                               */
    int32_t device;       /* CUDA device ordinal the context lives on               */
} kvs_config;

typedef struct {
    uint64_t append_launches;     /* kernels launched by kvs_append                          */
    uint64_t append_skipped;      /* kvs_append calls on sharing layers (no launch)          */
    uint64_t attention_launches;  /* split-K kernels launched                                */
    uint64_t combine_launches;    /* combine kernels launched                                */
    uint64_t kv_bytes_read;       /* 2*B*Hkv*n*D*elem summed over attention calls            */
    uint64_t kv_bytes_appended;   /* 2*B*Hkv*n_new*D*elem summed over launched appends       */
    uint64_t prefill_launches;    /* tensor-core prefill kernels launched                    */
    uint64_t evict_launches;      /* kvs_evict calls that launched                           */
    uint64_t search_launches;     /* kernels launched by kvs_layer_distances / kvs_mean_cosine */
    uint64_t fused_appends;       /* kvs_decode_step calls whose append rode in the split-K kernel */
} kvs_stats_t;

/* Tuning knobs for kvs_set_option.  Defaults are chosen by the library. */
typedef enum {
    KVS_OPT_MAX_CTAS = 0,   /* upper bound on thread blocks of the split-K kernel; 0 = auto  */
    KVS_OPT_KERNEL = 1,     /* 0 = auto, 1 = scalar-FMA path, 2 = grouped tensor-core path   */
    KVS_OPT_EARLY_START = 2,/* 1 (default): kernels are launched so that they may start while
                               the previous kernel on the stream drains, and prefetch K/V rows
                               that nothing in flight writes; they wait for the previous kernel
                               before reading q, newly appended rows, or writing anything.
                               0: plain stream-ordered launches.  Results are identical.      */
    KVS_OPT_REPLAY = 3,     /* 1: launches also read a device-side growth counter, so that a
                               recorded decode step can be replayed as a CUDA graph (see
                               kvs_replay_advance).  0 (default): lengths come from the host only. */
    KVS_OPT_HOST_CHUNKS = 4,/* kvs_step_host: number of pieces (1..8, default 4) the layers are cut
                               into for overlapping the host copies with the kernels.            */
    KVS_OPT_WAIT_LIMIT_US = 6,   /* limit of every wait inside the split-K kernels in microseconds (100 ..
                               10 000 000, default 2 000 000); on expiry the kernel gives up, see KVS_ERR_TIMEOUT */
    KVS_OPT_FINISH_IN_KERNEL = 5 /* 1 (default): when a call has at least as many (sequence, kv-head) units as
                               thread blocks, no unit is cut into more than two pieces and the split-K
                               kernel merges them itself (the block that holds a unit's first piece reads
                               the second, which the next block finished early in the same launch): one
                               launch per call instead of two.  0: always the separate combine kernel. */
} kvs_option;

/* ---- life cycle ------------------------------------------------------------ */

/* Create a context.  cfg: host.  *out receives the context.  The strategy
 * starts as the identity (no layer shares).  No CUDA call is made here.
 * Errors: INVALID_ARG for NULLs, non-positive sizes, Hq % Hkv != 0, group size
 * above 8 (or 3, 5, 6, 7 with fp32 storage), head_dim not in {64,128}, unknown dtype. */
kvs_status kvs_create(const kvs_config* cfg, kvs_ctx** out);

/* Destroy a context.  Frees host tables only; the caller's buffers are untouched.
 * The caller must have synchronised any stream that still runs work of this ctx. */
kvs_status kvs_destroy(kvs_ctx* ctx);

/* Install the sharing strategy (Section 3: a list saying which layers' KV caches
 * are replaced by which other layers').  share_map: host, n_layers entries;
 * share_map[l] == l means layer l computes its own cache, share_map[l] == s < l
 * means layer l uses the cache of layer s.  The paper always replaces the layer
 * nearer the output by the one nearer the input (Section 3.1), so s > l is
 * rejected with BAD_SHARE_MAP, as is s < 0.  Chains are legal and are followed
 * to the layer that computes its own cache.  Slots are numbered densely in
 * layer order over the layers that compute their own cache.
 * STATE unless every slot is empty (the strategy is fixed before inference).
 * Changes the required pool size: call before kvs_required_bytes/kvs_bind_memory;
 * a context that already has memory bound must be re-bound afterwards.          */
kvs_status kvs_set_share_map(kvs_ctx* ctx, const int32_t* share_map);

/* Bytes the caller must provide: pool = n_slots * 2 planes, workspace = split-K
 * partial results, a status word and staging for kvs_step_host.  Both host out. */
kvs_status kvs_required_bytes(const kvs_ctx* ctx, size_t* pool_bytes, size_t* workspace_bytes);

/* Hand the context its device memory.  pool, workspace: device, 256-byte
 * aligned, at least the sizes kvs_required_bytes reported (else OOM).  The pool
 * is zero-filled on the default stream and the call waits for that, so that
 * rows past a slot's length never hold non-finite bit patterns.  Queries device
 * properties; CUDA errors give KVS_ERR_CUDA.  Resets all slot lengths to 0.    */
kvs_status kvs_bind_memory(kvs_ctx* ctx, void* pool, size_t pool_bytes,
                           void* workspace, size_t workspace_bytes);

/* Forget every cached token (all slot lengths become 0).  Host-side only. */
kvs_status kvs_reset(kvs_ctx* ctx);

/* Forget the newest tokens: every slot that holds more than n_tokens rows is cut back to n_tokens
 * (the paper has no counterpart; generation only ever grows a cache, this is the roll-back a caller
 * needs to drop tokens it decides not to keep, or to run the same decode steps again).  Host-side
 * only, no launch: the rows stay in the pool and are overwritten by later appends.  Kernels already
 * queued keep the lengths they were launched with.  Not between the replays of a recorded step and
 * their kvs_replay_commit.  Errors: INVALID_ARG for n_tokens < 0; STATE if a slot that would be cut
 * has had rows evicted (its units differ in length).                                              */
kvs_status kvs_truncate(kvs_ctx* ctx, int32_t n_tokens);

/* ---- the hot path ------------------------------------------------------------ */

/* Store the new tokens' keys and values of one layer (Section 3.2; a layer whose
 * cache is replaced computes no KV -- caption of Table 1).
 *   layer computes its own cache: k, v are device pointers to
 *       [batch][n_new][n_kv_heads][head_dim] of the storage type; their rows are
 *       copied bit for bit to rows len .. len+n_new-1 of the layer's slot and the
 *       slot length grows by n_new.  One kernel launch on `stream`.
 *   layer's cache is replaced: returns KVS_OK at once; no launch, no length
 *       change, k and v are not read and may be NULL.
 * Errors: STATE before kvs_bind_memory; INVALID_ARG for a bad layer, batch < 1,
 * batch > max_batch, n_new < 1, NULL k/v on an own-cache layer, or a batch that
 * differs from the one the slot already holds rows for; CAPACITY if
 * len + n_new > max_seq.                                                        */
kvs_status kvs_append(kvs_ctx* ctx, int32_t layer, const void* k, const void* v,
                      int32_t batch, int32_t n_new, void* stream);

/* Attention of one layer's queries over the cache the layer uses (its own slot,
 * or its source layer's slot as it stands now -- Section 3.2: the source ran
 * earlier in the same forward pass, so its newest token is included):
 *   out[b][hq][:] = sum_j softmax_j(scale * q[b][hq] . K[b][hq/G][j]) V[b][hq/G][j]
 * over all n cached rows j, no mask, G = n_q_heads / n_kv_heads.
 *   q:   device, [batch][n_q_heads][head_dim], storage type
 *   out: device, [batch][n_q_heads][head_dim], float32
 * Launches the split-K kernel and the combine kernel on `stream`; partial
 * results go through the bound workspace, so calls on one context must not
 * overlap on the GPU (one stream, or full event ordering: see the conventions above).
 * Errors: STATE before kvs_bind_memory or when the slot is empty; INVALID_ARG
 * for a bad layer, NULLs, batch < 1 or batch > the batch the slot was filled for. */
kvs_status kvs_decode_attention(kvs_ctx* ctx, int32_t layer, const void* q, float* out,
                                int32_t batch, void* stream);

/* One decode step of one layer: kvs_append of one token (n_new = 1) followed by
 * kvs_decode_attention, with the same arguments, layouts, results and errors as those two
 * calls in that order (Section 3.2; on a layer whose cache is replaced k and v are not read and
 * may be NULL, and nothing is appended).
 *   q: device, [batch][n_q_heads][head_dim];  k, v: device, [batch][1][n_kv_heads][head_dim];
 *   out: device, float32 [batch][n_q_heads][head_dim]
 * On a computing layer whose slot nothing was evicted from no
 * append kernel is launched: the split-K kernel stores the new row itself -- the thread block
 * whose share of the rows ends a (sequence, kv-head) unit writes that unit's row to the slot just
 * before it fetches the tile that holds it -- so the step is two launches instead of three.  k and
 * v must stay valid until the call's work on `stream` has run.  Cached bits and output are those
 * of the two separate calls, bit for bit.  Otherwise the two calls are made as they are.        */
kvs_status kvs_decode_step(kvs_ctx* ctx, int32_t layer, const void* q, const void* k, const void* v,
                           float* out, int32_t batch, void* stream);

/* Prefill attention of one layer (Section 3.2: the strategy is applied to the prefill pass
 * as it is to generation).  The n_q queries per head are the newest n_q positions of the cache
 * the layer uses (its own slot, or its source layer's), i.e. call it after kvs_append has
 * stored those positions' K/V (on a sharing layer: after the source layer's append).  Causal
 * mask (the paper does not restate it; this is the usual decoder mask): query i sees rows
 * 0 .. n - n_q + i of the n cached rows.  Works for a whole prompt (n == n_q) and for a later
 * chunk of it (n > n_q).
 *   q:   device, [batch][n_q][n_q_heads][head_dim], storage type, 16-byte aligned
 *   out: device, [batch][n_q][n_q_heads][head_dim], float32
 * bf16 storage: one 4-byte clear and one tcgen05 tensor-core kernel on `stream`.  fp32 storage (the
 * small configuration): one plain fp32 kernel, a warp per query.  A slot rows were evicted from:
 * STATE.  Other errors as kvs_decode_attention; n_q > n: INVALID_ARG.                             */
kvs_status kvs_prefill_attention(kvs_ctx* ctx, int32_t layer, const void* q, float* out,
                                 int32_t batch, int32_t n_q, void* stream);

/* Keep only some rows of a layer's cache (the mechanics of combining layer sharing with an
 * intra-layer compression method, Section 4.4 and the reproduction appendix: each layer's cache
 * is sparsified in turn, and a layer that shares uses the sparsified cache of its source as it
 * is).  Which rows survive is the outside method's decision; this call only applies it.
 *   layer:  must compute its own cache (INVALID_ARG for a sharing layer); every layer that shares
 *           it sees the change, because they read the same slot
 *   keep:   device, int32 [batch][n_kv_heads][keep_stride]; the first n_keep[b*Hkv+h] entries of a
 *           unit are the row indices to keep, strictly ascending, each below the unit's length
 *   n_keep: host, int32 [batch * n_kv_heads], each in [1, current length of the unit]
 * The kept rows move to the front of the unit in order, bit for bit; afterwards the units of the
 * slot may differ in length ("ragged").  Appends then extend every unit at its own end,
 * kvs_decode_attention uses each unit's own length, kvs_seq_len reports the longest unit and
 * kvs_unit_len one unit; kvs_prefill_attention refuses a ragged slot (STATE).  One copy and two
 * kernels on `stream`.  A list that is not ascending or out of range cannot be seen by the host:
 * the kernel skips the offending entries and sets the device status word to KVS_ERR_INVALID_ARG.
 * Errors: STATE before bind or on an empty slot; INVALID_ARG for bad sizes or batch != cached batch. */
kvs_status kvs_evict(kvs_ctx* ctx, int32_t layer, const int32_t* keep, const int32_t* n_keep,
                     int32_t keep_stride, int32_t batch, void* stream);

/* Rows cached for sequence b, kv-head h of the slot `layer` reads. */
kvs_status kvs_unit_len(const kvs_ctx* ctx, int32_t layer, int32_t b, int32_t h, int32_t* len);

/* ---- the data-parallel reductions of strategy searching (Section 3.1, Algorithm 1) -------- */

/* Euclidean distances between the KV caches of every pair of layers.  The caches currently in
 * the pool play the calibration run: the first `batch` cached sequences are the samples.  Per
 * layer, keys and values are averaged over the samples, each flattened, and laid end to end
 * (reading of the averaging step of Section 3.1 / Algorithm 1: mean-K flattened, then mean-V
 * flattened, one vector per layer); dist[i][j] is the 2-norm of
 * the difference of layers i and j's vectors (a sharing layer has its source's cache: distance 0).
 *   dist: device, float32 [n_layers][n_layers], symmetric, zero diagonal.
 * Reads every cached element once: per slab of positions (sized so that the slab's sample means,
 * which pass through the workspace, stay in L2) one kernel averages the samples and one adds the
 * squared differences of every pair of cache slots; the averaging of the next slab is launched
 * behind it so that it starts beside it (a programmatic dependent launch on `stream`: no other
 * stream is used); two last kernels sum, take roots and expand slots to layers.  Not during
 * stream capture.
 * Sorting the pairs (descending, as the search does) is left to the caller.
 * Errors: STATE unless every slot holds the same non-zero number of rows and none is ragged, and while
 * `stream` is being captured; INVALID_ARG for batch > cached batch or more than 80 layers.                                */
kvs_status kvs_layer_distances(kvs_ctx* ctx, int32_t batch, float* dist, void* stream);

/* Cosine similarity of two models' averaged output representations: a and b are device tensors
 * [n_samples][dim] of the context's storage type (8-byte aligned, dim even); each is averaged
 * over the samples and *out (device, float32) receives cos(mean a, mean b).  Two kernels.       */
kvs_status kvs_mean_cosine(kvs_ctx* ctx, const void* a, const void* b, int32_t n_samples, int64_t dim,
                           float* out, void* stream);

/* ---- replaying a recorded decode step (CUDA graphs) ------------------------------------------
 * Slot lengths are host-side numbers baked into each launch, so a recorded launch would repeat
 * the same step.  With KVS_OPT_REPLAY = 1 every kvs_append / kvs_decode_attention launch also
 * adds a device-side counter to the lengths it was recorded with, and kvs_replay_advance
 * (record it as the last call of the step) adds one to that counter.  Each replay of
 * [append + attention for every layer, kvs_replay_advance] then appends one row further along and
 * attends over one row more: it is the next decode step (its inputs are read from the same device
 * buffers, which the caller refills between replays).  The thread blocks launched stay as
 * recorded; the split of the rows among them follows the grown length.
 *   - kvs_replay_advance only records something while `stream` is being captured; called on a
 *     stream that is not capturing it does nothing, so the same step function can first be run
 *     eagerly (an ordinary step) and then recorded.
 *   - While a stream is being captured, calls do their host bookkeeping as usual: the context's
 *     lengths advance as if the recorded step had run once.
 *   - After the recorded step has run `times_run` times in all (graph launches; if it was also
 *     run eagerly before capture with the counter at zero, those runs are ordinary steps and are
 *     not counted), call kvs_replay_commit(ctx, times_run, stream): the host lengths catch up
 *     (times_run - 1 more rows) and the counter is cleared on `stream`.  Make no eager call on
 *     the context between the first replay and the commit.
 *   - One-token decode steps only; every computing layer must append exactly once per step
 *     (kvs_append or kvs_decode_step).
 *   - A replay that would pass max_seq appends nothing for that layer and sets the device status
 *     word to KVS_ERR_CAPACITY; kvs_replay_commit returns CAPACITY instead of advancing.
 * Errors: STATE unless bound and KVS_OPT_REPLAY is 1; INVALID_ARG for times_run < 1.            */
kvs_status kvs_replay_advance(kvs_ctx* ctx, void* stream);
kvs_status kvs_replay_commit(kvs_ctx* ctx, int32_t times_run, void* stream);

/* One whole decode step from HOST buffers: for every layer in order, append the
 * layer's new token (own-cache layers only) and run its attention.
 *   q_host:   host, [n_layers][batch][n_q_heads][head_dim], storage type
 *   k_host, v_host: host, [n_layers][batch][1][n_kv_heads][head_dim], storage type
 *             (entries of sharing layers are not copied to the device)
 *   out_host: host, [n_layers][batch][n_q_heads][head_dim], float32
 * Copies inputs host->device into the workspace staging area, runs the layers on
 * `stream`, copies the result device->host, and waits until all of it is done.  The
 * copies run on two extra streams owned by the context (created at the first call,
 * together with a few events) in chunks of layers (KVS_OPT_HOST_CHUNKS), so that they overlap the
 * layers of the neighbouring chunks.
 * Pinned host memory makes the copies asynchronous; pageable memory also works.
 * h2d_bytes / d2h_bytes (host, may be NULL) receive the bytes copied.
 * Errors: as kvs_append / kvs_decode_attention; nothing is launched on an error
 * found before the first copy.                                                  */
kvs_status kvs_step_host(kvs_ctx* ctx, const void* q_host, const void* k_host, const void* v_host,
                         float* out_host, int32_t batch, void* stream,
                         uint64_t* h2d_bytes, uint64_t* d2h_bytes);

/* kvs_decode_attention for callers that have no scratch memory to give and may not
 * allocate any.  (The paper has no counterpart to this call; it exists for the users of
 * this library described below.)
 *
 * Who needs it: code that runs after a serving engine has handed all of the GPU's free memory
 * to its own pools and forbids further cudaMalloc (which would also stall the device); and code
 * in a plug-in or callback that is given tensors but no allocator.  Such callers still pass the
 * inputs and outputs (q, out, and the context whose pool holds K/V); what they cannot provide is
 * the scratch for split-K partial results.
 *
 * What it does: exactly what kvs_decode_attention does, with the same kernels and the same
 * result bit for bit, except that the partial results and the device status word live in a
 * fixed 2 MiB array inside the library image instead of the bound workspace.  The call
 * allocates nothing and frees nothing, on the device or through any library.
 *   - Every GPU that loads the library holds those 2 MiB until the process exits.
 *   - Limit: (batch * n_kv_heads + blocks launched) * group * (head_dim + 2) * 4 bytes of partial
 *     results, rounded up twice to 256 bytes, must fit in 2 MiB less 33 KiB (a status word and
 *     8192 per-unit hand-over flags at a fixed place); batch * n_kv_heads <= 8192.  The 7B shape at
 *     batch 8 needs 0.3 MiB, the 32q/8kv shape at batch 64 1.7 MiB.  Larger calls return
 *     KVS_ERR_SCRATCH_LIMIT and launch nothing.
 *   - The device address of the array is looked up once per GPU as part of kvs_bind_memory's
 *     per-device set-up (that look-up is also when the driver places the array on the GPU, so it
 *     happens where allocating is still allowed); the call itself makes no runtime query.
 *   - All calls, from all contexts and streams, share the one array, and it keeps the previous
 *     call's contents.  The call itself clears the status word; the hand-over flags are zero
 *     when the library is loaded and every launch leaves them zero again; nothing else must
 *     start at zero.  Two calls that overlap on the GPU race on the partial results: order
 *     them on one stream or with events.
 *   - The call is a plain stream-ordered launch and stays out of the context's launch
 *     bookkeeping, so it may be issued on another stream than the context's other calls, provided
 *     that stream waits (event) for the kernels that append the rows the call is to see; the other
 *     calls need not wait for it.  It reads the slot lengths as they stand on the host at the call.
 *   device_status: device pointer to an int32 (4-byte aligned, else INVALID_ARG) that receives 0,
 *     KVS_ERR_TIMEOUT if a bounded wait inside the kernel ran out, or (only under KVS_OPT_REPLAY)
 *     KVS_ERR_CAPACITY if a replayed launch passed max_seq; may be NULL (the word inside the array
 *     is used and is not readable by the caller).  It is written on `stream`; read it after
 *     synchronising.
 * Other arguments, layouts and errors: as kvs_decode_attention.                              */
kvs_status kvs_decode_attention_static(kvs_ctx* ctx, int32_t layer, const void* q, float* out,
                                       int32_t batch, void* stream, int32_t* device_status);

/* ---- introspection (index and layout checks are exact) ----------------------- */

kvs_status kvs_num_slots(const kvs_ctx* ctx, int32_t* n_slots);
kvs_status kvs_slot_of_layer(const kvs_ctx* ctx, int32_t layer, int32_t* slot);
/* Tokens visible to `layer` now (the length of the slot it reads; of its longest unit if ragged). */
kvs_status kvs_seq_len(const kvs_ctx* ctx, int32_t layer, int32_t* len);
/* Rows between consecutive (sequence, head) units of a plane. */
kvs_status kvs_row_stride(const kvs_ctx* ctx, int32_t* rows);
/* Byte offset into the pool of plane (slot, kv), kv = 0 for K, 1 for V. */
kvs_status kvs_plane_offset(const kvs_ctx* ctx, int32_t slot, int32_t kv, size_t* offset);
kvs_status kvs_stats(const kvs_ctx* ctx, kvs_stats_t* stats);
/* Reads the device status word (waits for the default stream's prior work on it):
 * 0 = no device-side problem; KVS_ERR_TIMEOUT = a bounded wait inside a kernel ran
 * out and the kernel returned early (its output is then undefined).             */
kvs_status kvs_last_device_status(kvs_ctx* ctx, int32_t* device_status);
/* Set the device status word back to 0 on `stream` (it is otherwise cleared only by kvs_bind_memory),
 * together with the per-unit hand-over flags a launch that gave up may have left raised: the way
 * back to a usable context after KVS_ERR_TIMEOUT (the output of the launch that gave up is lost). */
kvs_status kvs_clear_device_status(kvs_ctx* ctx, void* stream);
/* Failure-detection self-test of the attention kernels themselves (the paper has no counterpart).
 * Runs kvs_decode_attention with the same arguments, except that the producer of the thread block that
 * owns the middle tile of the call arms that tile's barrier and then withholds its K/V copies: the wait
 * for the tile runs out after KVS_OPT_WAIT_LIMIT_US (set it to a few milliseconds first), the block's
 * warps hand the give-up to one another, the producer waits for the copies it did issue, other blocks
 * that depend on this one give up in turn, and the launch ends normally with the device status word at
 * KVS_ERR_TIMEOUT and `out` undefined.  Nothing traps or faults, every wait on the way is bounded, and
 * kvs_clear_device_status brings the context back.  Same errors as kvs_decode_attention.               */
kvs_status kvs_selftest_stalled_copy(kvs_ctx* ctx, int32_t layer, const void* q, float* out, int32_t batch, void* stream);
/* Failure-detection self-test (the paper has no counterpart; every wait inside the pipelined kernels
 * is bounded, and this call shows the give-up path working on the device at hand without disturbing
 * anything).  Launches a one-warp kernel in which one thread waits, for at most limit_us
 * microseconds (1 .. 1 000 000), on a barrier that nothing ever arrives at, through the same bounded
 * wait the attention kernels use.  The wait runs out, the kernel sets the device status word to
 * KVS_ERR_TIMEOUT and returns normally; no copy is in flight, nothing traps, the context stays usable.
 * The call waits for the kernel; *waited_ns (host, may be NULL) receives how long the wait lasted on
 * the GPU.  Afterwards kvs_last_device_status reports KVS_ERR_TIMEOUT until kvs_clear_device_status.
 * Errors: STATE before kvs_bind_memory; INVALID_ARG for a limit out of range.                      */
kvs_status kvs_selftest_wait_timeout(kvs_ctx* ctx, uint32_t limit_us, uint64_t* waited_ns, void* stream);
/* Per-block timeline of the attention kernels (the paper has no counterpart; the library compiled with
 * -DKVS_TRACE only, STATE otherwise).  Between kvs_trace_begin and kvs_trace_end every attention call of the
 * context (kvs_decode_attention, kvs_decode_step, ...) writes 160 rows of 32 uint64 words to `buffer` (device,
 * 8-byte aligned, caller-owned), call after call, until `bytes` are used up: row b < 148 holds the GPU's
 * nanosecond timer as thread block b of the split-K kernel saw it at entry [0], when its producer's / its
 * consumers' wait for the previous kernel returned [1] / [2], when the first tile had arrived [3], when the
 * tiles of its k-th piece were done [4 + 2k] and the piece was merged and written [5 + 2k] (k < 8), when the
 * consumers ended [20], the number of pieces [21], when the producer began to wait [22], and the SM the
 * block ran on [23]; rows 150 and
 * 151 hold entry [0], end of wait [1] and end [2] of the first and the last block of the combine kernel
 * (zero when the call launched none).  kvs_trace_end stops the recording and reports the calls recorded.   */
kvs_status kvs_trace_begin(kvs_ctx* ctx, void* buffer, size_t bytes);
kvs_status kvs_trace_end(kvs_ctx* ctx, int32_t* launches_recorded);
/* Self-test of the bounds-checking build (the library compiled with -DKVS_DEBUG_BOUNDS, in which every
 * global offset the kernels compute is checked against the buffer it must fall in; the paper has no
 * counterpart).  Launches one kernel that hands the check an offset outside its buffer WITHOUT touching
 * memory; afterwards kvs_last_device_status reports KVS_ERR_BOUNDS, which shows that a real violation
 * would be recorded.  In a normal build the checks are compiled out: STATE, nothing is launched.   */
kvs_status kvs_selftest_bounds(kvs_ctx* ctx, void* stream);
kvs_status kvs_set_option(kvs_ctx* ctx, int32_t option, int32_t value);
/* How the last kvs_decode_attention call was decomposed: thread blocks launched,
 * rows per tile, and 1 or 2 for the scalar / tensor-core kernel.                */
kvs_status kvs_last_launch(const kvs_ctx* ctx, int32_t* ctas, int32_t* tile_rows, int32_t* kernel);
const char* kvs_status_string(kvs_status s);

/* ---- measurement support ------------------------------------------------------ */

/* Stream `bytes` (a non-zero multiple of 32768) from device memory `src` through the same
 * bulk-copy / shared-memory ring the attention kernel uses and fold them into
 * a checksum written to *checksum (device, 8 bytes).  Gives the read bandwidth
 * this staging scheme reaches when no arithmetic competes with it.  `device`
 * is the ordinal `src` lives on.  One launch on `stream`.                       */
kvs_status kvs_read_roof(const void* src, size_t bytes, uint64_t* checksum, int32_t device,
                         void* stream);

#ifdef __cplusplus
}
#endif
#endif /* KVS_H_ */
