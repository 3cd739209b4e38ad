/*
 * tensair.h - C ABI of the SGNS / DASGD hot path on one GPU.
 *
 * The library trains W logical replicas of a skip-gram negative-sampling (SGNS) word-embedding
 * model that live in one GPU's memory and exchange sparse gradient messages the way the Model
 * operator of Algorithm 1 does:
 *
 *   tensair_train_batch     train(msg), mini-batch branch of Algorithm 1: gradient calculation at
 *                           the snapshot theta_t (Eq. 1), local gradient application, then "send":
 *                           the sparse gradient message is filed for every other replica.
 *   tensair_apply_messages  train(msg), gradient branch of Algorithm 1: gradient application of the
 *                           messages another replica sent, in the order Section 3.1 fixes (after
 *                           the local step, received gradients one by one).
 *
 * Conventions for every call
 *   - Return value: TENSAIR_OK (0) or a negative TENSAIR_E* code; nothing throws or aborts across
 *     this boundary.  tensair_strerror() names a code, tensair_last_error() gives detail.
 *   - "device pointer" means memory of the GPU named in tensair_config.device; "host pointer" means
 *     ordinary process memory (pinned or pageable).
 *   - All GPU work is enqueued on the stream given at tensair_init, in call order (inside one call the
 *     library may fork part of the work onto internal streams and join it again before the call's
 *     last kernel; to the caller's stream the call is one ordered piece of work - what it has done is
 *     done when the stream has passed the call; part of it may have started earlier).  Calls are
 *     asynchronous unless stated; a context must be used from one thread at a time.
 *   - The library allocates no device memory: tables, message pool and scratch are caller-owned and
 *     must stay valid until tensair_destroy.
 *
 * Layouts
 *   - Tables: replica r owns 2*V rows of row_stride floats, input (centre-word) rows [0,V) followed
 *     by output (context-word) rows [V,2V); replicas are consecutive.  Only the first d floats of a
 *     row are meaningful.  A "row id" in [0,2V) names a row of this unified table.  Table entries must be
 *     finite: the kernels widen fp32 to fp64 by a bit manipulation that is exact for every finite value
 *     (subnormals and zeros included) but reads an infinity or a NaN as a finite number, so a table that has
 *     diverged to non-finite values gives unspecified (finite or not) results instead of propagating NaNs.
 *   - Sparse gradient message (the payload of Algorithm 1's send_gradients; Section 4 notes that a
 *     word-embedding mini-batch changes few of the model's variables, so only touched rows travel):
 *     a row count n, n strictly ascending row ids, n delta rows (already scaled by -lr).  Applying
 *     it is table[id] += delta, one fp32 addition per element.
 */
#ifndef TENSAIR_H
#define TENSAIR_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define TENSAIR_API __attribute__((visibility("default")))
#else
#define TENSAIR_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tensair_ctx tensair_ctx;
typedef struct tensair_schedule tensair_schedule;

/* How the batch loss L(X, theta) of Eq. 1 combines the per-pair losses (the paper does not say). */
enum { TENSAIR_SUM = 0, TENSAIR_MEAN = 1 };

enum {
    TENSAIR_OK = 0,
    TENSAIR_EINVAL = -1,    /* bad argument or unsupported configuration */
    TENSAIR_ENOMEM = -2,    /* a caller-provided buffer is too small */
    TENSAIR_ECUDA = -3,     /* a CUDA call failed; see tensair_last_error */
    TENSAIR_EBADTOKEN = -4, /* a batch held a token id outside [0,V) */
    TENSAIR_EPENDING = -5,  /* a message slot still has undelivered recipients */
    TENSAIR_ENOTFOUND = -6, /* the requested message is no longer held */
    TENSAIR_ETIMEOUT = -7,  /* a bounded wait inside a kernel ran out (a warp's own bulk copies did not land);
                               the batch it belonged to is incomplete */
    TENSAIR_EBOUNDS = -8    /* an index checked on the device was outside its array (checked builds), or a merged
                               message outgrew its slot; the access was skipped, nothing was written out of place */
};

/* Model, batch and exchange shape (Algorithm 1's constructor arguments plus the SGNS shape). */
typedef struct tensair_config {
    uint32_t V;               /* vocabulary size, 2 <= V <= 2^30 */
    uint32_t d;               /* embedding dimension, multiple of 4, 4 <= d <= 1024 */
    uint32_t window;          /* symmetric context window w, 1 <= w <= 16 */
    uint32_t k;               /* negatives per pair, 1 <= k <= 64 */
    uint32_t batch;           /* maximum centre tokens per mini-batch */
    uint32_t W;               /* logical replicas ("Model instances"), 1 <= W <= 256 */
    float lr;                 /* learning rate alpha of Eq. 1 */
    uint32_t max_grad_buffer; /* Algorithm 1's maxGradBuffer m, 1..8: a replica sends after every m-th of its batches */
    uint32_t max_delay;       /* messages are delivered 0..max_delay whole steps after their origin step */
    uint32_t row_stride;      /* floats between consecutive rows; 0 = d rounded up to a multiple of 8 */
    uint64_t seed;            /* key of the counter-based generator (negatives, delays, seeded init) */
    int32_t device;           /* CUDA device ordinal */
    uint32_t reduction;       /* TENSAIR_SUM: L(X) = sum of the pair losses; TENSAIR_MEAN: their mean over the batch's pairs */
} tensair_config;

typedef struct tensair_sizes {
    uint64_t tables_bytes;    /* W * 2V * row_stride * 4 */
    uint64_t pool_bytes;      /* W * (max_delay + 1) message slots of worst-case size */
    uint64_t scratch_bytes;   /* sort buffers, gradient scalars, partial sums, sampler table, counts */
    uint32_t row_stride;      /* the stride the library will use */
    uint32_t max_pairs;       /* pairs of a full batch: 2*w*batch - w*(w+1) when batch > w */
    uint32_t max_rows;        /* most rows a sent message can have (the capacity of a pool slot): distinct input rows
                                 <= min(m * batch, V) plus distinct output rows <= min(m * contributions, V),
                                 m = max_grad_buffer */
    uint32_t reserved;
} tensair_sizes;

/* Caller-owned device memory and stream.  All three pointers must be 256-byte aligned. */
typedef struct tensair_buffers {
    void* tables;
    uint64_t tables_bytes;
    void* pool;
    uint64_t pool_bytes;
    void* scratch;
    uint64_t scratch_bytes;
    void* stream;             /* cudaStream_t; NULL = the legacy default stream */
} tensair_buffers;

typedef struct tensair_msg_info {
    uint32_t n_rows;          /* rows in the message */
    uint32_t n_in_rows;       /* of which input rows (ids < V) */
    uint32_t n_pairs;         /* (centre, context) pairs of the batch */
    uint32_t slot;            /* pool slot the message occupies */
    uint64_t pool_offset;     /* byte offset of that slot in the pool */
} tensair_msg_info;

/* One entry of a receiver's delivery log. */
typedef struct tensair_delivery {
    uint64_t origin_step;     /* step at which the sender computed the gradient */
    uint64_t sender;
    uint64_t due_step;        /* origin_step + delay */
    uint64_t applied_at;      /* step argument of the apply call that delivered it */
    uint64_t staleness;       /* |G_i u G_j| - |G_i n G_j| of Section 3.1 */
} tensair_delivery;

/* Sizes the caller must allocate for a configuration.  No GPU is touched. */
TENSAIR_API int tensair_workspace_bytes(const tensair_config* cfg, tensair_sizes* out);

/*
 * Constructor of Algorithm 1 for all W replicas at once: every replica starts from the same model
 * (data parallelism as Section 2.2 describes it: identical initial replicas, disjoint data).
 *   counts_host   host, uint64[V] unigram counts for the count^0.75 negative sampler, or NULL = all 1.
 *                 Counts must be >= 1.  They also seed the running counts that train_batch increments.
 *   init_in_host  host, float[V*d] dense input rows, or NULL = seeded U(-0.5/d, 0.5/d).
 *   init_out_host host, float[V*d] dense output rows, or NULL = zeros.
 * Host arrays are read during the call only.  Synchronous.  The context borrows `bufs`.
 */
TENSAIR_API int tensair_init(const tensair_config* cfg, const tensair_buffers* bufs, const uint64_t* counts_host,
                 const float* init_in_host, const float* init_out_host, tensair_ctx** out);

/*
 * The same constructor for a job whose replicas are spread over several processes, one GPU each - the paper's
 * own placement: data parallelism with one Model instance per worker (Section 2.2) that sends each gradient to
 * every other instance (Section 3, "Stream Processing"; Algorithm 1, send_gradients).  The job has world_W
 * replicas with global ids 0..world_W-1; this context holds the tables of cfg->W of them, global ids
 * first_replica .. first_replica + cfg->W - 1.  Every process keeps the delivery schedule of the whole job (it
 * is a function of the seed) and a pool slot for every message in flight of every replica, local or not, so a
 * received message is applied from this GPU's own memory by the same kernels.  What differs from tensair_init:
 *   - negative draws, delivery delays and routing use the replica's global id, so the job computes what one
 *     process holding all world_W replicas computes, bit for bit (given the same batches per global replica);
 *   - `replica` arguments of the calls that touch tables (train, apply, read/write embeddings, snapshots, pending,
 *     delivery log) stay local indices 0..cfg->W-1; calls that name a message (tensair_read_message,
 *     tensair_message_buffers, tensair_commit_message) and tensair_shadow_apply take global ids;
 *   - per step, after the local tensair_train_batch calls: move every remote replica's message into the buffers
 *     tensair_message_buffers names (any transport: an NCCL broadcast or all-gather straight into the pool),
 *     tensair_commit_message each, then tensair_apply_messages for the local replicas and tensair_shadow_apply
 *     for the others.
 * tensair_workspace_bytes_sharded sizes the pool for world_W senders.  With world_W > cfg->W max_grad_buffer
 * must be 1 (TENSAIR_EINVAL otherwise): buffered gradients are merged only inside one process.
 * world_W == cfg->W and first_replica == 0 is tensair_init.
 */
TENSAIR_API int tensair_workspace_bytes_sharded(const tensair_config* cfg, uint32_t world_W, tensair_sizes* out);
TENSAIR_API int tensair_init_sharded(const tensair_config* cfg, const tensair_buffers* bufs, const uint64_t* counts_host,
                                     const float* init_in_host, const float* init_out_host, uint32_t first_replica,
                                     uint32_t world_W, tensair_ctx** out);

/* Where the message of (global sender, batch_index) lives in this context's pool (device pointers). */
typedef struct tensair_msg_view {
    uint32_t* ids;            /* device, uint32[max_rows]: the message's row ids, ascending */
    float* delta;             /* device, float[max_rows * row_stride]: its delta rows, row m at m * row_stride */
    uint32_t max_rows;        /* capacity of both arrays in rows */
    uint32_t row_stride;      /* floats between consecutive delta rows */
    uint64_t ids_offset;      /* byte offsets of the two arrays in the pool buffer given at init */
    uint64_t delta_offset;
    uint64_t header_offset;   /* byte offset of the slot's header: uint32 n_rows, uint32 n_in_rows (written on the
                                 device by the kernels that build the message; valid once the stream passed them) */
} tensair_msg_view;
/*
 * The "wire" of send_gradients (Algorithm 1) between processes.  Host-only, no synchronisation.
 *   local sender   the slot holding the message tensair_train_batch built for batch_index (TENSAIR_ENOTFOUND if
 *                  it is no longer held): the source of a send, valid once the stream has passed that call.
 *   remote sender  the slot the message must be received into; TENSAIR_EPENDING while the slot's previous
 *                  message still has local recipients (apply them first).  Write the first n_rows ids and
 *                  n_rows * row_stride floats in stream order, then call tensair_commit_message.
 */
TENSAIR_API int tensair_message_buffers(tensair_ctx* ctx, uint32_t sender, uint64_t batch_index, tensair_msg_view* out);
/* Row counts of a LOCAL replica's message (what a sender announces before its rows travel).  Synchronises. */
TENSAIR_API int tensair_message_rows(tensair_ctx* ctx, uint32_t replica, uint64_t batch_index, uint32_t* n_rows,
                                     uint32_t* n_in_rows);
/*
 * Files the received message of a REMOTE sender for this context's replicas (and books it for the others), as
 * tensair_train_batch does for a local one: writes the slot's header, builds the message's bucket index
 * (asynchronously on the context's stream, after whatever the stream already holds) and enters it in the delivery
 * schedule.  n_in_rows = how many of the ids are input rows (< V).  TENSAIR_EPENDING as for tensair_train_batch.
 */
TENSAIR_API int tensair_commit_message(tensair_ctx* ctx, uint32_t sender, uint64_t batch_index, uint32_t n_rows,
                                       uint32_t n_in_rows);
/*
 * The same with the header write and the bucket index enqueued on `stream` (a cudaStream_t of the context's device;
 * NULL = the context's stream) instead of the context's stream: for a caller that receives messages on a
 * communication stream of its own while the context's stream keeps training (Section 3.1: a Model goes on computing
 * while gradients arrive).  The entry in the delivery schedule is made at once, on the host, so the order of
 * these calls relative to the train and apply calls is what fixes delivery order and staleness, as before.  The
 * caller orders the streams: `stream` must have received the rows before this call, and the context's stream must
 * wait for `stream` (an event recorded after this call) before the first apply call at which the message is due.
 */
TENSAIR_API int tensair_commit_message_on(tensair_ctx* ctx, uint32_t sender, uint64_t batch_index, uint32_t n_rows,
                                          uint32_t n_in_rows, void* stream);
/*
 * Book-keeping of a REMOTE receiver: marks what is due for it at `step` (or everything, drain != 0) as applied,
 * which the process holding that replica does for real.  Keeps slot reuse and the staleness of Section 3.1
 * (which needs every replica's set of applied gradients) exact in every process.  Host-only.
 */
TENSAIR_API int tensair_shadow_apply(tensair_ctx* ctx, uint32_t receiver, uint64_t step, int drain, uint32_t* n_applied);

/*
 * Resuming a run in flight (Section 3.3: models are saved and loaded; here the run around them as well).  What a run
 * consists of: the tables and the message pool (the caller's device buffers: copy them as they are, after
 * tensair_sync), and what the library keeps - the running unigram counts, the sampler table in use, the messages
 * buffered under max_grad_buffer > 1 (their count; the rows are in the pool) and the delivery schedule with its
 * pending deliveries, applied-gradient sets and logs.  tensair_save_state writes the library's part to host memory
 * (dst NULL: only *bytes, the size needed; TENSAIR_ENOMEM if capacity is short); tensair_load_state puts it into a
 * context made by tensair_init / tensair_init_sharded with the SAME configuration (TENSAIR_EINVAL otherwise), after
 * which the caller restores its copies of tables and pool.  The resumed run then computes, bit for bit, what the
 * uninterrupted run computes.  Both synchronise.
 */
TENSAIR_API int tensair_save_state(tensair_ctx* ctx, void* host_dst, uint64_t capacity, uint64_t* bytes);
TENSAIR_API int tensair_load_state(tensair_ctx* ctx, const void* host_src, uint64_t bytes);

/* Frees host state only; synchronises the stream first. */
TENSAIR_API void tensair_destroy(tensair_ctx* ctx);

/*
 * One mini-batch on one replica (Algorithm 1, train, mini-batch branch; Eq. 1):
 *   pairs      every (centre position q, context position c) with 0 < |q-c| <= window inside the
 *              batch's own n_tokens tokens, in (q ascending, c ascending) order;
 *   negatives  k per pair from the counter-based sampler; one equal to the pair's context word is dropped;
 *   gradient   of the SGNS loss of the whole batch (sum or mean of the pair losses, see `reduction`) at
 *              the replica's tables as they are when the call starts (nothing is updated mid-batch);
 *              dot products, sigmoids and row sums are taken in fp64 from the fp32 tables;
 *   message    one delta row fp32(-lr * gradient) per touched row, ids ascending;
 *   local GA   the message is applied to the replica at once (staleness 0);
 *   send       it is filed for every other replica at step batch_index + delay(batch_index, replica, j).
 *              With max_grad_buffer = m > 1 (Algorithm 1: gradients are accumulated and sent when their count
 *              reaches maxGradBuffer) only every m-th batch of a replica sends: the sum of its last m
 *              messages over the union of their rows, each row's deltas added in fp32 in the order they
 *              were computed; tensair_read_message then holds only for those batch indices.
 * tokens_dev   device, int32[n_tokens], borrowed until the stream has passed this call; n_tokens <= batch.  They are
 *              read in stream order (whatever the stream holds before this call may still be writing them), unless
 *              the knob "early_prepare" of tensair_tune is 2: the caller then vouches that tokens_dev is complete
 *              when the call is made (batches resident in device memory, a copy already waited for), and the
 *              library samples and sorts a batch (of up to "early_prepare_max_items" sort items) on an internal stream
 *              ahead of the batch's turn on the caller's stream - beside the batches before it or beside the message
 *              application.  Results do not depend on the knobs.
 * batch_index  the global step t of this batch (< 2^32); it selects the random draws and the message slot.
 * loss_out     host, nullable.  Non-NULL: receives the sum of the batch's pair losses and the call synchronises.
 * info         host, nullable.  Non-NULL: filled, and the call synchronises.
 * A token id outside [0,V) leaves tables, counts and pool untouched and raises TENSAIR_EBADTOKEN at
 * the next synchronising call (this one if loss_out or info is given); batches enqueued after the
 * bad one and before that call are dropped too.
 * TENSAIR_EPENDING: the slot of step batch_index - (max_delay+1) still has undelivered recipients
 * (tensair_apply_messages was not called for them).
 */
TENSAIR_API int tensair_train_batch(tensair_ctx* ctx, uint32_t replica, const int32_t* tokens_dev, uint32_t n_tokens,
                        uint64_t batch_index, double* loss_out, tensair_msg_info* info);

/* Same step with the batch in HOST memory: copies tokens_host to the device first (asynchronously if the memory is
 * pinned).  Host memory is complete when the call is made, so (unless the knob "early_prepare" is 0) the copy, the
 * sampling and the sort of the batch run on an internal stream ahead of the batch's turn on the caller's stream.
 * tokens_host must stay valid until the stream passes. */
TENSAIR_API int tensair_train_batch_host(tensair_ctx* ctx, uint32_t replica, const int32_t* tokens_host, uint32_t n_tokens,
                             uint64_t batch_index, double* loss_out, tensair_msg_info* info);

/*
 * The same step for a mini-batch that the W replicas share (Section 4.3: the (x, y) pairs are spread over the
 * Model instances by a hash partitioner keyed by the word x).  Every replica is handed the same tokens_dev and
 * trains the pairs whose centre word is routed to it:
 *     route(x) = (Philox4x32-10(counter = (x, 0, 0, 4 << 24), key = seed).word0 * W) >> 32     (tensair_route).
 * The W calls compute disjoint parts of one mini-batch gradient: the pair index p, the negative draws (replica
 * tag 0 in their counter) and, for TENSAIR_MEAN, the divisor are those of the whole batch, so the W messages add
 * up to the message one model computes from the batch; their input rows are disjoint.  The running unigram
 * counts take each token once, from the replica that owns it.  info->n_pairs is the pair count of the whole
 * batch.  Arguments, asynchrony and errors as for tensair_train_batch; the taps tensair_read_negatives and
 * tensair_read_scalars are defined only for the pairs the replica owns.
 */
TENSAIR_API int tensair_train_batch_routed(tensair_ctx* ctx, uint32_t replica, const int32_t* tokens_dev,
                                           uint32_t n_tokens, uint64_t batch_index, double* loss_out,
                                           tensair_msg_info* info);
/* The replica that owns centre word `token` under the routing above (host only). */
TENSAIR_API int tensair_route(uint64_t seed, uint32_t W, uint32_t token, uint32_t* replica);

/*
 * The same step for callers that may not allocate device memory when they train - a plug-in that is
 * handed its tables and message pool by a host application with a fixed memory plan, or a service
 * thread that must stay out of the allocator.  (The paper has no counterpart: this is an addition of
 * this library.)  Arguments, results, error codes and the filing of the message are those of
 * tensair_train_batch, and the result is bit-identical to it.  The difference: part of the per-batch
 * working memory is not taken from the scratch buffer given at tensair_init but from a fixed 32 MiB
 * array inside the library image, which every GPU that loads the library reserves until the process
 * exits.  Taken from the array: the two sort buffers, the sorted terms, the partial centre gradients and
 * losses per position, the radix histograms, the segment starts, the long-row lists and their chunk
 * partials.  Still in the context's scratch (it exists anyway, tensair_init needed it): the error word,
 * the loss, the running counts, the sampler table, the per-contribution row ids and gradient scalars.
 * The call allocates nothing on the device, neither directly nor through a library.
 *   - Only for max_grad_buffer = 1 (TENSAIR_EINVAL otherwise).
 *   - TENSAIR_ENOMEM (with the sizes in tensair_last_error) when the context's configuration needs
 *     more of that memory than the array holds.  With I = 2 * batch + pairs * (k+1) sort items
 *     (pairs = 2 * window * batch - window * (window+1)) the need is about
 *       I * (8 + 8 + 16)  +  2 * batch * row_stride * 8  +  (I / 32 + 2) * row_stride * 8  +  I / 4  bytes
 *     (sort buffers and terms; partial centre gradients, two per position; chunk partials; lists and
 *     histograms): e.g. V = 20,000, d = 64, window 5, k = 5, batch 1,024 needs 4 MiB; batch 8,192 at
 *     d = 300, k = 15 needs 180 MiB and is refused.
 *   - The first call on a device looks up the array's device address (once per device, with that device
 *     current, under a lock, so first calls from several threads are safe); where the driver loads modules
 *     lazily, it may reserve the array's 32 MiB only then, so the device's free memory can change at that first
 *     call and at no later one.  Make that first call before any stream capture begins.
 *   - All calls, from all contexts of the process on one GPU, share the one array.  It keeps the last
 *     call's contents; the call clears what it needs to be zero itself.  Two calls that may overlap on
 *     the GPU (contexts on different streams) race on it: serialise them.
 *   - The parity taps tensair_read_negatives and tensair_read_scalars work after this call as well.
 */
TENSAIR_API int tensair_train_batch_static(tensair_ctx* ctx, uint32_t replica, const int32_t* tokens_dev,
                                           uint32_t n_tokens, uint64_t batch_index, double* loss_out,
                                           tensair_msg_info* info);

/*
 * Algorithm 1, train, gradient branch, for one receiver: applies every pending message whose due step
 * is <= step, in (origin step, sender) order - the order in which Section 3.1 has a Model work off
 * the gradients that arrived while it was busy.  Call it for step t after every replica has run
 * tensair_train_batch for step t.  A second call for the same (replica, step) applies nothing.
 * n_applied: host, nullable.
 */
TENSAIR_API int tensair_apply_messages(tensair_ctx* ctx, uint32_t replica, uint64_t step, uint32_t* n_applied);

/*
 * tensair_apply_messages(replica, step) for every replica of the context, as one pass over their tables: a
 * message due for several of them at this step is read from memory once and added to each (the replicas share
 * one GPU's memory, so the gradient application that every Model instance repeats - Section 4.2 notes that it is
 * not distributed - shares its reads here).  Per replica the messages are applied in
 * the same (origin step, sender) order, so tables and delivery logs are bit-identical to the per-replica calls.
 * n_applied: host, nullable: deliveries made, summed over the replicas.
 */
TENSAIR_API int tensair_apply_step(tensair_ctx* ctx, uint64_t step, uint32_t* n_applied);

/* End of a run: delivers everything still pending, per receiver in (due step, origin step, sender)
 * order, so that all replicas have applied the same gradients.  n_applied: host, nullable. */
TENSAIR_API int tensair_drain(tensair_ctx* ctx, uint32_t* n_applied);

/* Rebuilds the negative sampler's alias table from the running unigram counts (initial counts plus
 * every token trained on so far).  The table is built on the device, asynchronously on the context's
 * stream, bit-identical to what tensair_build_alias_host gives for the same counts.  (With the knob
 * "device_alias_build" = 0 of tensair_tune the counts are read back, one host thread builds the table
 * and the call synchronises.) */
TENSAIR_API int tensair_update_sampler(tensair_ctx* ctx);

/* The loss of the most recent tensair_train_batch* call without waiting for it: enqueues, on the context's
 * stream, a copy of the batch loss (sum of the pair losses) into host_dst (host, double; pinned memory for the
 * copy to be asynchronous).  The value is there once the stream has passed the copy, e.g. after tensair_sync;
 * one synchronisation per step can so serve the losses of all replicas.  host_dst must stay valid until then. */
TENSAIR_API int tensair_read_loss_async(tensair_ctx* ctx, double* host_dst);

/* Waits for the stream; returns and clears a pending device-side error: TENSAIR_EBADTOKEN, TENSAIR_ETIMEOUT or
 * TENSAIR_EBOUNDS (the gravest of those raised; tensair_last_error names all). */
TENSAIR_API int tensair_sync(tensair_ctx* ctx);

/* Copies rows [row0, row0+nrows) of a replica's input (which=0) or output (which=1) table into
 * host_dst as dense float[nrows*d].  Synchronises.  (For this model "prediction" is this lookup.) */
TENSAIR_API int tensair_read_embeddings(tensair_ctx* ctx, uint32_t replica, int which, uint32_t row0, uint32_t nrows,
                            float* host_dst);
/* The reverse copy (restore from a dump).  Synchronises. */
TENSAIR_API int tensair_write_embeddings(tensair_ctx* ctx, uint32_t replica, int which, uint32_t row0, uint32_t nrows,
                             const float* host_src);

/*
 * Drift metric of Section 4.3 (Table 1): how far an embedding row has moved between two points of the
 * stream, as the cosine difference 1 - cos(a, b) of the row now (a) and in an earlier snapshot (b).
 *   tensair_snapshot_rows      copies rows [row0, row0+nrows) of a table into snap_dev, device float[nrows*d] dense.
 *   tensair_cosine_difference  writes 1 - (a.b) / (|a| |b|) per row into out_dev, device float[nrows]; dot and
 *                              norms in fp64; two zero rows give 0, one zero row gives 1.
 * Both are asynchronous on the context's stream; the buffers are the caller's.
 */
TENSAIR_API int tensair_snapshot_rows(tensair_ctx* ctx, uint32_t replica, int which, uint32_t row0, uint32_t nrows,
                                      float* snap_dev);
TENSAIR_API int tensair_cosine_difference(tensair_ctx* ctx, uint32_t replica, int which, uint32_t row0, uint32_t nrows,
                                          const float* snap_dev, float* out_dev);

/*
 * The rows that drifted most, as Table 1 of Section 4.3 lists the words whose embeddings moved most: the
 * min(k, nrows) largest entries of diff_dev (device float[nrows], e.g. what tensair_cosine_difference wrote),
 * largest first, the smaller index first among equal values.  Values are ranked by the total order of their
 * fp32 bit patterns (-NaN < -inf < ... < -0 < +0 < ... < +inf < +NaN), so the result is defined for any input
 * and is bit-exact.  ids_dev (device uint32[k], indices into diff_dev) and vals_dev (device float[k]) are the
 * caller's; entries past min(k, nrows) are left alone; *n_out (host, nullable) receives min(k, nrows).
 * k <= 4096, else TENSAIR_EINVAL.  Asynchronous on the context's stream; works in the context's scratch, which
 * stream order keeps apart from the training calls.
 */
TENSAIR_API int tensair_top_drifted(tensair_ctx* ctx, const float* diff_dev, uint32_t nrows, uint32_t k, uint32_t* ids_dev,
                                    float* vals_dev, uint32_t* n_out);

/* ---- parity taps (synchronous; for tests and diagnostics) ---- */

/* Raw negative draws of the last train_batch call: host uint32[n_pairs*k] (nullable); n_pairs nullable. */
TENSAIR_API int tensair_read_negatives(tensair_ctx* ctx, uint32_t* host_neg, uint32_t* n_pairs);
/* Gradient scalars g[p][0..k] of the last train_batch call (dropped negatives read 0): host double[n_pairs*(k+1)]. */
TENSAIR_API int tensair_read_scalars(tensair_ctx* ctx, double* host_g);
/* Message of (replica, batch_index) while its slot has not been reused: n_rows (nullable), ids
 * host uint32[n_rows] (nullable), delta host float[n_rows*d] dense (nullable). */
TENSAIR_API int tensair_read_message(tensair_ctx* ctx, uint32_t replica, uint64_t batch_index, uint32_t* n_rows,
                         uint32_t* host_ids, float* host_delta);
/* Sampler state: any of thresh uint32[V], alias uint32[V], counts uint64[V] (host, nullable). */
TENSAIR_API int tensair_read_sampler(tensair_ctx* ctx, uint32_t* thresh, uint32_t* alias, uint64_t* counts);
/* Delivery log of one receiver, oldest first: up to max_records entries into host `out`; n receives the count held. */
TENSAIR_API int tensair_read_delivery_log(tensair_ctx* ctx, uint32_t replica, uint64_t max_records, tensair_delivery* out,
                              uint64_t* n);
/* Messages filed for a receiver and not yet applied. */
TENSAIR_API int tensair_pending(tensair_ctx* ctx, uint32_t replica, uint64_t* n);
/* Kernels launched by this context so far. */
TENSAIR_API uint64_t tensair_kernel_launches(const tensair_ctx* ctx);

/* Per-kernel timing.  While enabled, every kernel launch is bracketed by a pair of CUDA events on the
 * context's stream (a few microseconds of overhead per launch, so do not time whole steps with it on).
 * tensair_profile_read synchronises, writes one record per kernel kind (up to max_kinds; n_kinds =
 * how many kinds exist) with the launches and summed device time since the previous read, and
 * forgets them. */
typedef struct tensair_kernel_time {
    char name[32];
    uint64_t launches;
    double total_ms;
} tensair_kernel_time;
TENSAIR_API int tensair_profile(tensair_ctx* ctx, int enable);
/* Launch-shape knobs for sweeps (process-wide; results do not depend on them): "forward_rows" = 8 or 16
 * output rows reduced together by a warp of the forward kernel (0 = default), "forward_blocks_per_sm"
 * = resident blocks per multiprocessor the forward grid is sized for (0 = default),
 * "reduce_blocks_per_sm" / "apply_blocks_per_sm" = blocks per multiprocessor of the row-sum / message-apply grids,
 * "fuse_apply" = 0 applies the messages due for a receiver one launch each instead of in one pass,
 * "fused_blocks_per_sm" = blocks per multiprocessor of that pass, "overlap_sort" = 0 keeps the sort of a batch on the caller's stream instead of an internal second stream,
 * "overlap_long_rows" = 0 keeps the sums of the rows with many contributions, the message's bucket index and the
 * loss sum on the caller's stream instead of beside the short-row sums on the second stream,
 * "device_alias_build" = 0 makes tensair_update_sampler build the table on the host,
 * "early_prepare" = 0 / 1 / 2: a batch's sampling and sort run ahead of its turn on an internal third stream never /
 * when its tokens come from host memory (default) / also for device tokens, which the caller then vouches are complete
 * when the call is made; "early_prepare_max_items" = largest batch, in sort items (two per token plus window pairs
 * times (k+1)), that is prepared ahead (default 2^20: larger batches gain nothing from it). */
TENSAIR_API int tensair_tune(const char* name, int value);
TENSAIR_API int tensair_profile_read(tensair_ctx* ctx, uint32_t max_kinds, tensair_kernel_time* out, uint32_t* n_kinds);

TENSAIR_API const char* tensair_strerror(int code);
TENSAIR_API const char* tensair_last_error(const tensair_ctx* ctx);

/* The device-side error word.  Kernels never trap: one that meets bad input or gives up a bounded wait sets a bit
 * of a sticky word in the scratch buffer and skips its work; the next synchronising call turns the word into a code.
 *   bit 0 (1)  a token id outside [0,V)                          -> TENSAIR_EBADTOKEN
 *   bit 1 (2)  a wait for a warp's own bulk copies ran out        -> TENSAIR_ETIMEOUT
 *   bit 2 (4)  checked build: an index outside its array         -> TENSAIR_EBOUNDS
 *   bit 3 (8)  a merged message outgrew its slot                  -> TENSAIR_EBOUNDS
 * tensair_error_of_flags gives the code a value of the word stands for (host only, no context needed).
 * tensair_raise_error_flags ORs bits into a context's word from the host, as a kernel would have: a hook for testing
 * a caller's error handling without making a GPU misbehave.  Synchronises.
 *
 * Checked build: compiled with -DTENSAIR_BOUNDS (`python -m paper_2211_10280_b200.build --bounds`, which writes
 * libtensair_checked.so beside the normal library), every index that a kernel computes from data - row ids against
 * the table, message rows against the slot, sort positions, list and scratch offsets - is compared with its bound
 * before use; a violation raises bit 2 and skips the access.  tensair_checked_build() says which build is loaded. */
TENSAIR_API int tensair_checked_build(void);
TENSAIR_API int tensair_error_of_flags(uint32_t flags);
TENSAIR_API int tensair_raise_error_flags(tensair_ctx* ctx, uint32_t flags);

/* ---- host-only pieces, usable without a GPU ---- */

/* Walker/Vose alias table over weights count^0.75 (counts NULL = all 1): host in, host out. */
TENSAIR_API int tensair_build_alias_host(const uint64_t* counts, uint32_t V, uint32_t* thresh, uint32_t* alias);
/* Philox4x32-10: counter[4], key[2] -> out[4]. */
TENSAIR_API void tensair_philox4x32_10(const uint32_t counter[4], const uint32_t key[2], uint32_t out[4]);
/* Delivery delay, in whole steps, of the message (sender, step) to `receiver`: uniform in 0..max_delay. */
TENSAIR_API uint32_t tensair_delay(uint64_t seed, uint32_t max_delay, uint64_t step, uint32_t sender, uint32_t receiver);

/*
 * The delivery schedule and staleness bookkeeping on their own (the context owns one of these).
 * on_train   records that `replica` computed and locally applied gradient (replica, step) and files
 *            it for every other replica; TENSAIR_EPENDING if the slot it would reuse is still pending.
 * take_due   pops the receiver's deliveries with due step <= step in (origin step, sender) order (or,
 *            with drain != 0, all of them in (due, origin, sender) order), marks them applied at `step`
 *            (at their due step when draining) and writes up to max_records of them; n = how many popped.
 */
TENSAIR_API int tensair_schedule_create(uint32_t W, uint32_t max_delay, uint64_t seed, tensair_schedule** out);
TENSAIR_API void tensair_schedule_destroy(tensair_schedule* s);
TENSAIR_API int tensair_schedule_on_train(tensair_schedule* s, uint32_t replica, uint64_t step);
TENSAIR_API int tensair_schedule_take_due(tensair_schedule* s, uint32_t receiver, uint64_t step, int drain,
                              uint64_t max_records, tensair_delivery* out, uint64_t* n);
TENSAIR_API int tensair_schedule_pending(const tensair_schedule* s, uint32_t receiver, uint64_t* n);
/* The schedule's whole book-keeping as bytes (dst NULL: only *bytes, the size needed) and back; load accepts only what
 * a schedule of the same W, max_delay and seed saved (TENSAIR_EINVAL otherwise, nothing changed). */
TENSAIR_API int tensair_schedule_save(const tensair_schedule* s, void* dst, uint64_t capacity, uint64_t* bytes);
TENSAIR_API int tensair_schedule_load(tensair_schedule* s, const void* src, uint64_t bytes);

#ifdef __cplusplus
}
#endif
#endif /* TENSAIR_H */
