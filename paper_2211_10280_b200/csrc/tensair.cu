// C ABI of the library: context, workspace carving, the train / apply / drain calls and the parity taps.
#include "../../include/tensair.h"

#include <cstdio>
#include <algorithm>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "context.h"

using namespace tensair;

namespace {

int validate_config(const tensair_config* c) {
    if (!c) return TENSAIR_EINVAL;
    if (c->V < 2 || c->V > (1u << 30)) return TENSAIR_EINVAL;
    if (c->d < 4 || c->d > 1024 || c->d % 4) return TENSAIR_EINVAL;
    if (c->window < 1 || c->window > 16) return TENSAIR_EINVAL;
    if (c->k < 1 || c->k > 64) return TENSAIR_EINVAL;
    if (c->batch < 1 || c->batch > (1u << 22)) return TENSAIR_EINVAL;
    if (c->W < 1 || c->W > 256) return TENSAIR_EINVAL;
    if (c->max_grad_buffer < 1 || c->max_grad_buffer > (uint32_t)kMaxMerge) return TENSAIR_EINVAL;
    if (c->max_delay > 64) return TENSAIR_EINVAL;
    if (c->row_stride && (c->row_stride < c->d || c->row_stride % 4)) return TENSAIR_EINVAL;
    if (!(c->lr == c->lr)) return TENSAIR_EINVAL;
    if (c->device < 0 || c->device >= kMaxDevices) return TENSAIR_EINVAL;
    if (c->reduction > TENSAIR_MEAN) return TENSAIR_EINVAL;
    const uint64_t contrib = (uint64_t)pair_count(c->batch, c->window) * (c->k + 1);
    if (contrib + c->batch >= (1ull << 31)) return TENSAIR_EINVAL;
    return TENSAIR_OK;
}

void carve(const tensair_config& c, Carve& k) {
    k.stride = c.row_stride ? c.row_stride : (uint32_t)round_up(c.d, 8);
    k.max_pairs = pair_count(c.batch, c.window);
    k.max_contrib = k.max_pairs * (c.k + 1);
    k.max_items = 2 * c.batch + k.max_contrib;   // two input-row items per position, then the contributions
    k.max_rows = (c.batch < c.V ? c.batch : c.V) + (k.max_contrib < c.V ? k.max_contrib : c.V);
    // A sent message is the union of maxGradBuffer batch messages: up to m times the rows of one, capped by the tables.
    const uint64_t m_in = (uint64_t)c.max_grad_buffer * c.batch, m_out = (uint64_t)c.max_grad_buffer * k.max_contrib;
    k.slot_rows = (uint32_t)((m_in < c.V ? m_in : c.V) + (m_out < c.V ? m_out : c.V));
    k.max_long = k.max_items / kChunk + 1;
    k.max_chunks = 2 * (k.max_items / kChunk) + 2;
    uint64_t off = 0;
    auto take = [&off](uint64_t bytes) { const uint64_t at = off; off = round_up(off + bytes, 256); return at; };
    k.err = take(4);
    k.loss = take(8);
    k.long_counters = take(16);
    k.counts = take((uint64_t)c.V * 8);
    k.alias_tab = take((uint64_t)c.V * 8);
    k.tok = take((uint64_t)c.batch * 4);
    k.rows = take((uint64_t)k.max_contrib * 4);
    k.items_a = take((uint64_t)k.max_items * 8);
    k.items_b = take((uint64_t)k.max_items * 8);
    k.rec = take((uint64_t)k.max_contrib * sizeof(Rec));
    k.terms = take((uint64_t)k.max_items * sizeof(Rec));
    k.gin_pos = take((uint64_t)2 * c.batch * k.stride * 8);
    k.loss_pos = take((uint64_t)2 * c.batch * 8);
    k.hist = take((uint64_t)sort_hist_words(k.max_items) * 4);
    k.tile_counts = take((uint64_t)(heads_tiles(k.max_items) + 1) * 4);
    k.seg_start = take((uint64_t)(k.max_rows + 2) * 4);
    k.long_rows = take((uint64_t)k.max_long * sizeof(LongRow));
    k.chunk_items = take((uint64_t)k.max_chunks * sizeof(ChunkItem));
    k.partials = take((uint64_t)k.max_chunks * k.stride * 8);
    k.merge_counts = take((uint64_t)(bucket_count(c.V) + 1) * 4);
    k.topk = take(sizeof(TopkState));
    k.owner = take(c.batch);
    k.owned = take((uint64_t)c.batch * 4);
    k.n_owned = take(4);
    k.alias_state = take(sizeof(AliasState));
    k.alias_work = take(alias_work_bytes(c.V));
    // buffer sets of the batches prepared ahead of their turn: offsets inside a set, then the sets themselves
    {
        uint64_t in = 0;
        auto part = [&in](uint64_t bytes) { const uint64_t at = in; in = round_up(in + bytes, 256); return at; };
        k.set_err = part(4);
        k.set_tok = part((uint64_t)c.batch * 4);
        k.set_rows = part((uint64_t)k.max_contrib * 4);
        k.set_items_a = part((uint64_t)k.max_items * 8);
        k.set_items_b = part((uint64_t)k.max_items * 8);
        k.set_hist = part((uint64_t)sort_hist_words(k.max_items) * 4);
        k.set_bytes = in;
    }
    k.set_base = take((uint64_t)tensair_ctx::kPrepSets * k.set_bytes);
    k.total = off;
    k.bucket_off = kHeaderBytes;
    k.ids_off = round_up(k.bucket_off + (uint64_t)(bucket_count(c.V) + 1) * 4, 256);
    k.delta_off = round_up(k.ids_off + (uint64_t)k.slot_rows * 4, 256);
    k.slot_bytes = round_up(k.delta_off + (uint64_t)k.slot_rows * k.stride * 4, 256);
}

}  // namespace

namespace tensair {

int fail(tensair_ctx* ctx, cudaError_t e, const char* what) {
    if (ctx) ctx->last_error = std::string(what) + ": " + cudaGetErrorString(e);
    return TENSAIR_ECUDA;
}

// What a value of the device error word means.  Several bits may be set; the code is that of the gravest
// (an index out of bounds, then a wait that ran out, then bad input), the text names all of them.
int error_of_flags(uint32_t flags, std::string* text) {
    if (!flags) return TENSAIR_OK;
    std::string t;
    auto add = [&t](const char* what) { if (!t.empty()) t += "; "; t += what; };
    if (flags & kErrBounds) add("a checked index was outside its array (the access was skipped)");
    if (flags & kErrOverflow) add("a merged message had more rows than its slot holds");
    if (flags & kErrTimeout) add("a wait for a warp's own asynchronous copies ran out (the batch is incomplete)");
    if (flags & kErrBadToken) add("a batch held a token id outside [0,V)");
    if (flags & ~(kErrBounds | kErrOverflow | kErrTimeout | kErrBadToken)) add("unknown error bits");
    t += "; that batch and the batches after it were dropped";
    if (text) *text = t;
    if (flags & (kErrBounds | kErrOverflow)) return TENSAIR_EBOUNDS;
    if (flags & kErrTimeout) return TENSAIR_ETIMEOUT;
    if (flags & kErrBadToken) return TENSAIR_EBADTOKEN;
    return TENSAIR_ECUDA;
}

// Reads and clears the device error word after a synchronisation.
int collect(tensair_ctx* ctx) {
    TENSAIR_CUDA(ctx, cudaMemcpyAsync(&ctx->stage->err, ctx->at<uint32_t>(ctx->cv.err), 4, cudaMemcpyDeviceToHost, ctx->stream));
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (ctx->stage->err) {
        TENSAIR_CUDA(ctx, cudaMemsetAsync(ctx->at<uint32_t>(ctx->cv.err), 0, 4, ctx->stream));
        return error_of_flags(ctx->stage->err, &ctx->last_error);
    }
    return TENSAIR_OK;
}

}  // namespace tensair

namespace {

int upload_sampler(tensair_ctx* ctx, const uint64_t* counts_host) {
    const uint32_t V = ctx->cfg.V;
    std::vector<uint32_t> thresh(V), alias(V);
    build_alias_host(counts_host, V, thresh.data(), alias.data());
    std::vector<uint2> packed(V);
    for (uint32_t i = 0; i < V; ++i) packed[i] = make_uint2(thresh[i], alias[i]);
    TENSAIR_CUDA(ctx, cudaMemcpyAsync(ctx->at<uint2>(ctx->cv.alias_tab), packed.data(), (size_t)V * 8, cudaMemcpyHostToDevice, ctx->stream));
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return TENSAIR_OK;
}

// routed: the replica trains only the centre positions whose word the hash partitioner gives it (Section 4.3);
// pair indices, negative draws (replica tag 0) and the mean's denominator stay those of the whole batch.
// tok_host != nullptr: the batch is in host memory (complete when the call is made) and is copied to the device here.
int train_impl(tensair_ctx* ctx, uint32_t replica, const int32_t* tok_dev, uint32_t n, uint64_t batch_index,
               double* loss_out, tensair_msg_info* info, bool routed = false, const int32_t* tok_host = nullptr) {
    const tensair_config& c = ctx->cfg;
    const Carve& cv = ctx->cv;
    // maxGradBuffer = 1: the batch's message is built in its send slot and filed at once.  Otherwise it is built
    // in a buffer slot of the replica, and after every m-th batch the m buffered messages are summed into a send slot.
    const uint32_t m_buf = c.max_grad_buffer;
    const uint32_t me = ctx->gid(replica);   // the replica's id among all replicas of the job
    const uint32_t send_slot = ctx->sched->slot_of(me, batch_index);
    const bool sends = m_buf == 1 || ctx->buffered[replica] + 1 == m_buf;
    if (sends && m_buf > 1 && ctx->sched->slot_busy(send_slot)) return TENSAIR_EPENDING;
    if (m_buf == 1) {
        const int rc = ctx->sched->on_train(me, batch_index);
        if (rc != TENSAIR_OK) return rc;
    }
    const uint32_t slot = m_buf == 1 ? send_slot
                                     : ctx->world_W * (c.max_delay + 1) + replica * m_buf + ctx->buffered[replica];
    const uint32_t pairs = n >= 2 ? pair_count(n, c.window) : 0;
    const uint32_t contrib = pairs * (c.k + 1);
    const uint32_t n_items = pairs ? 2 * n + contrib : 0;
    uint32_t* err = ctx->at<uint32_t>(cv.err);
    float* table = ctx->table_of(replica);
    MsgHeader* hdr = ctx->slot_hdr(slot);
    // Eq. 1's alpha, divided by the number of pairs when the batch loss is the mean of the pair losses
    const double scale = c.reduction == TENSAIR_MEAN && pairs ? (double)c.lr / (double)pairs : (double)c.lr;

    uint8_t* owner = routed ? ctx->at<uint8_t>(cv.owner) : nullptr;
    uint32_t* owned = routed ? ctx->at<uint32_t>(cv.owned) : nullptr;
    uint32_t* n_owned = routed ? ctx->at<uint32_t>(cv.n_owned) : nullptr;
    // The sampling and the sort of a batch need only its tokens and the sampler table, not the model: with the tokens
    // known to be complete (host memory, or the caller's word for device memory) they run on a third stream into a
    // buffer set of their own, ahead of the batch's turn on the caller's stream - beside the kernels of the batches
    // before it or beside the message application - and the forward kernel then has the machine to itself.
    // It pays where a batch is bound by launch latency (measured: batch 256 0.130 -> 0.087 ms, batch 2,048 0.240 ->
    // 0.194 ms at d = 300, k = 5); for large batches the sort costs whatever it runs beside as much as it costs the
    // forward kernel, so those keep the sort beside their own forward kernel.
    const bool early = !routed && n_items && n_items <= (uint32_t)grid_shape().early_prepare_max_items && ctx->prep &&
                       (grid_shape().early_prepare >= 2 || (grid_shape().early_prepare == 1 && tok_host));
    const uint32_t* rows_of_batch = ctx->at<uint32_t>(cv.rows);
    item_t* sorted = nullptr;
    int set = -1;
    if (early) {
        set = ctx->next_set;
        ctx->next_set = (set + 1) % tensair_ctx::kPrepSets;
        // the set's previous batch must have read its sorted items; the sampler table must be the current one
        if (ctx->set_used[set]) TENSAIR_CUDA(ctx, cudaStreamWaitEvent(ctx->prep, ctx->ev_set_free[set], 0));
        if (ctx->sampler_rebuilt) TENSAIR_CUDA(ctx, cudaStreamWaitEvent(ctx->prep, ctx->ev_sampler, 0));
        uint32_t* batch_err = ctx->in_set<uint32_t>(set, cv.set_err);
        if (tok_host) {
            int32_t* staged = ctx->in_set<int32_t>(set, cv.set_tok);
            TENSAIR_CUDA(ctx, cudaMemcpyAsync(staged, tok_host, (size_t)n * 4, cudaMemcpyHostToDevice, ctx->prep));
            tok_dev = staged;
        }
        TENSAIR_CUDA(ctx, cudaMemsetAsync(batch_err, 0, 4, ctx->prep));
        uint32_t* rows = ctx->in_set<uint32_t>(set, cv.set_rows);
        TENSAIR_CUDA(ctx, launch_prepare(ctx->L_prep, tok_dev, n, ctx->shape, me, (uint32_t)batch_index, c.seed,
                                         ctx->at<uint2>(cv.alias_tab), rows, ctx->in_set<item_t>(set, cv.set_items_a),
                                         ctx->at<unsigned long long>(cv.counts), batch_err, nullptr, true, false));
        TENSAIR_CUDA(ctx, cudaEventRecord(ctx->ev_prepared[set], ctx->prep));
        TENSAIR_CUDA(ctx, launch_sort(ctx->L_prep, ctx->in_set<item_t>(set, cv.set_items_a), ctx->in_set<item_t>(set, cv.set_items_b),
                                      n_items, bits_for(2 * c.V), ctx->in_set<uint32_t>(set, cv.set_hist), &sorted));
        TENSAIR_CUDA(ctx, cudaEventRecord(ctx->ev_sorted[set], ctx->prep));
        ctx->last_prepared = set;
        rows_of_batch = rows;
        TENSAIR_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev_prepared[set], 0));
        TENSAIR_CUDA(ctx, launch_forward(ctx->L, tok_dev, n, ctx->shape, table, rows, ctx->at<Rec>(cv.rec),
                                         ctx->at<double>(cv.gin_pos), ctx->at<double>(cv.loss_pos), err, nullptr, nullptr,
                                         batch_err, false));
        TENSAIR_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev_sorted[set], 0));
        ctx->set_used[set] = true;
    } else {
    if (tok_host) {
        int32_t* staged = ctx->at<int32_t>(cv.tok);
        if (n) TENSAIR_CUDA(ctx, cudaMemcpyAsync(staged, tok_host, (size_t)n * 4, cudaMemcpyHostToDevice, ctx->stream));
        tok_dev = staged;
    }
    // A routed batch needs the owner of every centre word before anything else, and that kernel checks the token ids
    // as well; otherwise the prepare kernel checks them itself.  A batch with pairs has its tokens counted by the
    // first kernel of the message build (by then the whole batch is known to be valid), a shorter one here.
    if (routed || !n_items)
        TENSAIR_CUDA(ctx, launch_validate(ctx->L, tok_dev, n, c.V, err, owner, owned, n_owned, ctx->world_W, me, c.seed));
    TENSAIR_CUDA(ctx, launch_prepare(ctx->L, tok_dev, n, ctx->shape, routed ? 0u : me, (uint32_t)batch_index, c.seed,
                                     ctx->at<uint2>(cv.alias_tab), ctx->at<uint32_t>(cv.rows),
                                     ctx->at<item_t>(cv.items_a), ctx->at<unsigned long long>(cv.counts), err, owner,
                                     !routed && n_items, !n_items));
    }
    ctx->last_rows = rows_of_batch;
    if (n_items) {
        if (!early) {
        // The sort needs only the items written by the prepare kernel and the forward kernel does not
        // touch them: the two run side by side (the sort is latency-bound and leaves the machine idle).
        const bool fork = ctx->side && grid_shape().overlap_sort;
        if (fork) {
            TENSAIR_CUDA(ctx, cudaEventRecord(ctx->ev_fork, ctx->stream));
            TENSAIR_CUDA(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0));
        }
        TENSAIR_CUDA(ctx, launch_sort(fork ? ctx->L_side : ctx->L, ctx->at<item_t>(cv.items_a), ctx->at<item_t>(cv.items_b),
                                      n_items, bits_for(2 * c.V), ctx->at<uint32_t>(cv.hist), &sorted));
        TENSAIR_CUDA(ctx, launch_forward(ctx->L, tok_dev, n, ctx->shape, table, ctx->at<uint32_t>(cv.rows),
                                         ctx->at<Rec>(cv.rec), ctx->at<double>(cv.gin_pos), ctx->at<double>(cv.loss_pos), err,
                                         owned, n_owned));
        if (fork) {
            TENSAIR_CUDA(ctx, cudaEventRecord(ctx->ev_join, ctx->side));
            TENSAIR_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev_join, 0));
        }
        }
        TENSAIR_CUDA(ctx, launch_heads(ctx->L, sorted, n_items, c.V, ctx->at<uint32_t>(cv.tile_counts), hdr,
                                       ctx->slot_ids(slot), ctx->at<uint32_t>(cv.seg_start),
                                       ctx->at<uint32_t>(cv.long_counters), ctx->at<Rec>(cv.rec),
                                       ctx->at<Rec>(cv.terms), err, ctx->at<LongRow>(cv.long_rows),
                                       ctx->at<ChunkItem>(cv.chunk_items), tok_dev, n,
                                       ctx->at<unsigned long long>(cv.counts), owner));
        // the set's sorted items are dead once the heads kernels have gathered the terms
        if (early) TENSAIR_CUDA(ctx, cudaEventRecord(ctx->ev_set_free[set], ctx->stream));
        // The few rows with many contributions, the message's bucket index and the loss are small latency-bound
        // kernels; they touch nothing the short-row kernel writes, so they run beside it on the second stream.
        const bool beside = ctx->side && grid_shape().overlap_long_rows;
        const Launcher& L2 = beside ? ctx->L_side : ctx->L;
        if (beside) {
            TENSAIR_CUDA(ctx, cudaEventRecord(ctx->ev_fork, ctx->stream));
            TENSAIR_CUDA(ctx, cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0));
        }
        TENSAIR_CUDA(ctx, launch_reduce_long_rows(L2, ctx->at<Rec>(cv.terms), ctx->slot_ids(slot), ctx->at<uint32_t>(cv.seg_start),
                                                  ctx->at<double>(cv.gin_pos), table, ctx->slot_delta(slot), ctx->shape, scale,
                                                  ctx->at<uint32_t>(cv.long_counters), ctx->at<LongRow>(cv.long_rows),
                                                  ctx->at<ChunkItem>(cv.chunk_items), ctx->at<double>(cv.partials)));
        TENSAIR_CUDA(ctx, launch_bucket_index(L2, hdr, ctx->slot_ids(slot), ctx->slot_buckets(slot), c.V,
                                              ctx->at<double>(cv.loss_pos), n, ctx->at<double>(cv.loss), err, owner));
        TENSAIR_CUDA(ctx, launch_reduce_rows(ctx->L, ctx->at<Rec>(cv.terms), hdr, ctx->slot_ids(slot), ctx->at<uint32_t>(cv.seg_start),
                                             ctx->at<double>(cv.gin_pos), table, ctx->slot_delta(slot), ctx->shape, scale));
        if (beside) {
            TENSAIR_CUDA(ctx, cudaEventRecord(ctx->ev_join, ctx->side));
            TENSAIR_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, ctx->ev_join, 0));
        }
        // input rows last: they were the sources of every output-row sum
        TENSAIR_CUDA(ctx, launch_apply_rows(ctx->L, hdr, ctx->slot_ids(slot), ctx->slot_delta(slot), table, ctx->shape, 1));
    } else {
        TENSAIR_CUDA(ctx, cudaMemsetAsync(hdr, 0, sizeof(MsgHeader), ctx->stream));
        TENSAIR_CUDA(ctx, launch_bucket_index(ctx->L, hdr, ctx->slot_ids(slot), ctx->slot_buckets(slot), c.V));
        TENSAIR_CUDA(ctx, launch_loss_sum(ctx->L, ctx->at<double>(cv.loss_pos), n, ctx->at<double>(cv.loss), err, owner));
    }
    if (m_buf > 1) {
        ++ctx->buffered[replica];
        if (sends) {
            // Algorithm 1: the buffered gradients are sent once their count reaches maxGradBuffer
            MergeInputs in;
            in.count = m_buf;
            for (uint32_t b = 0; b < m_buf; ++b) {
                const uint32_t bs = ctx->world_W * (c.max_delay + 1) + replica * m_buf + b;
                in.ids[b] = ctx->slot_ids(bs);
                in.delta[b] = ctx->slot_delta(bs);
                in.buckets[b] = ctx->slot_buckets(bs);
            }
            TENSAIR_CUDA(ctx, launch_merge(ctx->L, in, ctx->slot_hdr(send_slot), ctx->slot_buckets(send_slot),
                                           ctx->slot_ids(send_slot), ctx->slot_delta(send_slot),
                                           ctx->at<uint32_t>(cv.merge_counts), ctx->shape, cv.slot_rows, err));
            const int rc = ctx->sched->on_train(me, batch_index);
            if (rc != TENSAIR_OK) return rc;
            ctx->buffered[replica] = 0;
        }
    }
    ctx->last_n = n;
    ctx->last_pairs = pairs;
    ctx->have_last = true;
    if (loss_out || info) {
        TENSAIR_CUDA(ctx, cudaMemcpyAsync(&ctx->stage->loss, ctx->at<double>(cv.loss), 8, cudaMemcpyDeviceToHost, ctx->stream));
        TENSAIR_CUDA(ctx, cudaMemcpyAsync(&ctx->stage->hdr, hdr, sizeof(MsgHeader), cudaMemcpyDeviceToHost, ctx->stream));
        const int st = collect(ctx);
        if (st != TENSAIR_OK) return st;
        if (loss_out) *loss_out = ctx->stage->loss;
        if (info) {
            info->n_rows = ctx->stage->hdr.n_rows;
            info->n_in_rows = ctx->stage->hdr.n_in_rows;
            info->n_pairs = pairs;
            info->slot = slot;
            info->pool_offset = (uint64_t)slot * cv.slot_bytes;
        }
    }
    return TENSAIR_OK;
}

int apply_due(tensair_ctx* ctx, uint32_t receiver, const std::vector<Due>& due) {
    // Messages are applied in the order given; up to kMaxStepMessages of them share one pass over the table.
    size_t at = 0;
    const size_t replica_floats = (size_t)2 * ctx->cfg.V * ctx->cv.stride;
    while (at < due.size()) {
        const size_t k = grid_shape().fuse_apply ? std::min(due.size() - at, (size_t)kMaxStepMessages) : 1;
        if (k == 1) {
            const Due& d = due[at];
            TENSAIR_CUDA(ctx, launch_apply(ctx->L, ctx->slot_hdr(d.slot), ctx->slot_ids(d.slot), ctx->slot_delta(d.slot),
                                           ctx->table_of(receiver), ctx->shape));
        } else {
            StepMessages f;
            f.count = (uint32_t)k;
            for (size_t i = 0; i < k; ++i) {
                const uint32_t slot = due[at + i].slot;
                f.ids[i] = ctx->slot_ids(slot);
                f.delta[i] = ctx->slot_delta(slot);
                f.buckets[i] = ctx->slot_buckets(slot);
                f.receivers[i] = 1u;
            }
            TENSAIR_CUDA(ctx, launch_apply_step(ctx->L, f, 1, ctx->table_of(receiver), replica_floats, ctx->shape, K_APPLY_FUSED));
        }
        at += k;
    }
    return TENSAIR_OK;
}

int copy_rows(tensair_ctx* ctx, uint32_t replica, int which, uint32_t row0, uint32_t nrows, float* host, bool to_host) {
    const tensair_config& c = ctx->cfg;
    if (replica >= c.W || (which != 0 && which != 1) || (uint64_t)row0 + nrows > c.V || (!host && nrows)) return TENSAIR_EINVAL;
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (!nrows) return TENSAIR_OK;
    float* dev = ctx->table_of(replica) + ((size_t)which * c.V + row0) * ctx->cv.stride;
    if (to_host)
        TENSAIR_CUDA(ctx, cudaMemcpy2D(host, (size_t)c.d * 4, dev, (size_t)ctx->cv.stride * 4, (size_t)c.d * 4, nrows, cudaMemcpyDeviceToHost));
    else
        TENSAIR_CUDA(ctx, cudaMemcpy2D(dev, (size_t)ctx->cv.stride * 4, host, (size_t)c.d * 4, (size_t)c.d * 4, nrows, cudaMemcpyHostToDevice));
    return TENSAIR_OK;
}

}  // namespace

extern "C" {

int tensair_workspace_bytes(const tensair_config* cfg, tensair_sizes* out) {
    return tensair_workspace_bytes_sharded(cfg, cfg ? cfg->W : 0, out);
}

int tensair_workspace_bytes_sharded(const tensair_config* cfg, uint32_t world_W, tensair_sizes* out) {
    const int rc = validate_config(cfg);
    if (rc != TENSAIR_OK || !out || world_W < cfg->W || world_W > 256) return TENSAIR_EINVAL;
    Carve cv;
    carve(*cfg, cv);
    out->row_stride = cv.stride;
    out->tables_bytes = (uint64_t)cfg->W * 2 * cfg->V * cv.stride * 4;
    // one slot per message in flight of every replica of the job, plus (maxGradBuffer > 1) the buffered messages
    // of the replicas that live here
    out->pool_bytes = ((uint64_t)world_W * (cfg->max_delay + 1) +
                       (cfg->max_grad_buffer > 1 ? (uint64_t)cfg->W * cfg->max_grad_buffer : 0)) * cv.slot_bytes;
    out->scratch_bytes = cv.total;
    out->max_pairs = cv.max_pairs;
    out->max_rows = cv.slot_rows;
    out->reserved = 0;
    return TENSAIR_OK;
}

int tensair_init(const tensair_config* cfg, const tensair_buffers* bufs, const uint64_t* counts_host,
                 const float* init_in_host, const float* init_out_host, tensair_ctx** out) {
    return tensair_init_sharded(cfg, bufs, counts_host, init_in_host, init_out_host, 0, cfg ? cfg->W : 0, out);
}

int tensair_init_sharded(const tensair_config* cfg, const tensair_buffers* bufs, const uint64_t* counts_host,
                         const float* init_in_host, const float* init_out_host, uint32_t first_replica,
                         uint32_t world_W, tensair_ctx** out) {
    tensair_sizes sz;
    if (!out || !bufs || tensair_workspace_bytes_sharded(cfg, world_W, &sz) != TENSAIR_OK) return TENSAIR_EINVAL;
    *out = nullptr;
    if ((uint64_t)first_replica + cfg->W > world_W) return TENSAIR_EINVAL;
    // buffered gradients are merged where they were computed; a job spread over processes sends every batch
    if (world_W > cfg->W && cfg->max_grad_buffer != 1) return TENSAIR_EINVAL;
    if (!bufs->tables || !bufs->pool || !bufs->scratch) return TENSAIR_EINVAL;
    if (((uintptr_t)bufs->tables | (uintptr_t)bufs->pool | (uintptr_t)bufs->scratch) & 255) return TENSAIR_EINVAL;
    if (bufs->tables_bytes < sz.tables_bytes || bufs->pool_bytes < sz.pool_bytes || bufs->scratch_bytes < sz.scratch_bytes)
        return TENSAIR_ENOMEM;
    if (counts_host)
        for (uint32_t i = 0; i < cfg->V; ++i) if (counts_host[i] < 1) return TENSAIR_EINVAL;
    DeviceGuard guard(cfg->device);
    if (!guard.ok) return TENSAIR_ECUDA;
    tensair_ctx* ctx = new (std::nothrow) tensair_ctx();
    if (!ctx) return TENSAIR_ENOMEM;
    ctx->cfg = *cfg;
    ctx->world_W = world_W;
    ctx->first = first_replica;
    carve(*cfg, ctx->cv);
    ctx->shape = Shape{cfg->V, cfg->d, cfg->d / 4, ctx->cv.stride, cfg->window, cfg->k, cfg->k + 1};
    ctx->stream = (cudaStream_t)bufs->stream;
    ctx->tables = (float*)bufs->tables;
    ctx->pool = (uint8_t*)bufs->pool;
    ctx->scratch = (uint8_t*)bufs->scratch;
    cudaDeviceProp prop;
    int status = TENSAIR_OK;
    auto bail = [&](int code) {
        delete ctx->sched;
        if (ctx->stage) cudaFreeHost(ctx->stage);
        if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
        if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
        if (ctx->side) cudaStreamDestroy(ctx->side);
        if (ctx->ev_call) cudaEventDestroy(ctx->ev_call);
        if (ctx->ev_sampler) cudaEventDestroy(ctx->ev_sampler);
        for (int i = 0; i < tensair_ctx::kPrepSets; ++i) {
            if (ctx->ev_prepared[i]) cudaEventDestroy(ctx->ev_prepared[i]);
            if (ctx->ev_sorted[i]) cudaEventDestroy(ctx->ev_sorted[i]);
            if (ctx->ev_set_free[i]) cudaEventDestroy(ctx->ev_set_free[i]);
        }
        if (ctx->prep) cudaStreamDestroy(ctx->prep);
        delete ctx;
        return code;
    };
    if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return bail(TENSAIR_ECUDA);
    ctx->L = Launcher{ctx->stream, &ctx->launches, prop.multiProcessorCount, &ctx->prof, cfg->device};
    ctx->L.lim = Limits{reinterpret_cast<uint32_t*>(ctx->scratch + ctx->cv.err), 2 * cfg->V, ctx->cv.slot_rows, ctx->cv.max_rows,
                        ctx->cv.max_items, ctx->cv.max_contrib, 2 * cfg->batch, ctx->cv.max_long, ctx->cv.max_chunks};
    if (cudaMallocHost((void**)&ctx->stage, sizeof(*ctx->stage)) != cudaSuccess) return bail(TENSAIR_ECUDA);
    ctx->sched = new Schedule(world_W, cfg->max_delay, cfg->seed);
    ctx->buffered.assign(cfg->W, 0);
    // The second stream carries small latency-bound kernels that run beside a long one on the caller's
    // stream; the highest priority lets their blocks in as soon as a slot is free.
    int prio_low = 0, prio_high = 0;
    if (cudaDeviceGetStreamPriorityRange(&prio_low, &prio_high) != cudaSuccess) return bail(TENSAIR_ECUDA);
    if (cudaStreamCreateWithPriority(&ctx->side, cudaStreamNonBlocking, prio_high) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) != cudaSuccess)
        return bail(TENSAIR_ECUDA);
    ctx->L_side = ctx->L;
    ctx->L_side.stream = ctx->side;
    if (cudaStreamCreateWithPriority(&ctx->prep, cudaStreamNonBlocking, prio_high) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_call, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_sampler, cudaEventDisableTiming) != cudaSuccess)
        return bail(TENSAIR_ECUDA);
    for (int i = 0; i < tensair_ctx::kPrepSets; ++i)
        if (cudaEventCreateWithFlags(&ctx->ev_prepared[i], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_sorted[i], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&ctx->ev_set_free[i], cudaEventDisableTiming) != cudaSuccess)
            return bail(TENSAIR_ECUDA);
    ctx->L_prep = ctx->L;
    ctx->L_prep.stream = ctx->prep;

    const uint32_t V = cfg->V, stride = ctx->cv.stride;
    const size_t replica_floats = (size_t)2 * V * stride;
    auto run = [&]() -> int {
        TENSAIR_CUDA(ctx, cudaMemsetAsync(ctx->scratch, 0, ctx->cv.total, ctx->stream));
        TENSAIR_CUDA(ctx, cudaMemsetAsync(ctx->pool, 0, sz.pool_bytes, ctx->stream));
        TENSAIR_CUDA(ctx, cudaMemsetAsync(ctx->tables, 0, replica_floats * 4, ctx->stream));
        if (init_in_host)
            TENSAIR_CUDA(ctx, cudaMemcpy2DAsync(ctx->tables, (size_t)stride * 4, init_in_host, (size_t)cfg->d * 4,
                                                (size_t)cfg->d * 4, V, cudaMemcpyHostToDevice, ctx->stream));
        else
            TENSAIR_CUDA(ctx, launch_init_input_table(ctx->L, ctx->tables, ctx->shape, cfg->seed));
        if (init_out_host)
            TENSAIR_CUDA(ctx, cudaMemcpy2DAsync(ctx->tables + (size_t)V * stride, (size_t)stride * 4, init_out_host,
                                                (size_t)cfg->d * 4, (size_t)cfg->d * 4, V, cudaMemcpyHostToDevice, ctx->stream));
        for (uint32_t r = 1; r < cfg->W; ++r)
            TENSAIR_CUDA(ctx, cudaMemcpyAsync(ctx->tables + r * replica_floats, ctx->tables, replica_floats * 4,
                                              cudaMemcpyDeviceToDevice, ctx->stream));
        std::vector<uint64_t> ones;
        const uint64_t* counts = counts_host;
        if (!counts) { ones.assign(V, 1); counts = ones.data(); }
        TENSAIR_CUDA(ctx, cudaMemcpyAsync(ctx->at<uint64_t>(ctx->cv.counts), counts, (size_t)V * 8, cudaMemcpyHostToDevice, ctx->stream));
        TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        return upload_sampler(ctx, counts);
    };
    status = run();
    if (status != TENSAIR_OK) return bail(status);
    *out = ctx;
    return TENSAIR_OK;
}

void tensair_destroy(tensair_ctx* ctx) {
    if (!ctx) return;
    DeviceGuard guard(ctx->cfg.device);
    cudaStreamSynchronize(ctx->stream);
    for (const Profiler::Span& sp : ctx->prof.spans) { cudaEventDestroy(sp.start); cudaEventDestroy(sp.stop); }
    for (cudaEvent_t e : ctx->prof.spare) cudaEventDestroy(e);
    if (ctx->stage) cudaFreeHost(ctx->stage);
    if (ctx->side) {
        cudaStreamSynchronize(ctx->side);
        cudaEventDestroy(ctx->ev_fork);
        cudaEventDestroy(ctx->ev_join);
        cudaStreamDestroy(ctx->side);
    }
    if (ctx->prep) {
        cudaStreamSynchronize(ctx->prep);
        cudaEventDestroy(ctx->ev_call);
        cudaEventDestroy(ctx->ev_sampler);
        for (int i = 0; i < tensair_ctx::kPrepSets; ++i) {
            cudaEventDestroy(ctx->ev_prepared[i]);
            cudaEventDestroy(ctx->ev_sorted[i]);
            cudaEventDestroy(ctx->ev_set_free[i]);
        }
        cudaStreamDestroy(ctx->prep);
    }
    delete ctx->sched;
    delete ctx;
}

int tensair_train_batch(tensair_ctx* ctx, uint32_t replica, const int32_t* tokens_dev, uint32_t n_tokens,
                        uint64_t batch_index, double* loss_out, tensair_msg_info* info) {
    if (!ctx || replica >= ctx->cfg.W || n_tokens > ctx->cfg.batch || (n_tokens && !tokens_dev) ||
        batch_index >= (1ull << 32))
        return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    return train_impl(ctx, replica, tokens_dev, n_tokens, batch_index, loss_out, info);
}

int tensair_train_batch_routed(tensair_ctx* ctx, uint32_t replica, const int32_t* tokens_dev, uint32_t n_tokens,
                               uint64_t batch_index, double* loss_out, tensair_msg_info* info) {
    if (!ctx || replica >= ctx->cfg.W || n_tokens > ctx->cfg.batch || (n_tokens && !tokens_dev) ||
        batch_index >= (1ull << 32))
        return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    return train_impl(ctx, replica, tokens_dev, n_tokens, batch_index, loss_out, info, true);
}

int tensair_train_batch_host(tensair_ctx* ctx, uint32_t replica, const int32_t* tokens_host, uint32_t n_tokens,
                             uint64_t batch_index, double* loss_out, tensair_msg_info* info) {
    if (!ctx || replica >= ctx->cfg.W || n_tokens > ctx->cfg.batch || (n_tokens && !tokens_host) ||
        batch_index >= (1ull << 32))
        return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    return train_impl(ctx, replica, nullptr, n_tokens, batch_index, loss_out, info, false, tokens_host);
}

int tensair_apply_messages(tensair_ctx* ctx, uint32_t replica, uint64_t step, uint32_t* n_applied) {
    if (!ctx || replica >= ctx->cfg.W) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    const std::vector<Due> due = ctx->sched->take_due(ctx->gid(replica), step, false);
    if (n_applied) *n_applied = (uint32_t)due.size();
    return apply_due(ctx, replica, due);
}

int tensair_apply_step(tensair_ctx* ctx, uint64_t step, uint32_t* n_applied) {
    if (!ctx) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    const uint32_t W = ctx->cfg.W;
    std::vector<std::vector<Due>> due(W);
    uint32_t total = 0;
    for (uint32_t r = 0; r < W; ++r) {
        due[r] = ctx->sched->take_due(ctx->gid(r), step, false);
        total += (uint32_t)due[r].size();
    }
    if (n_applied) *n_applied = total;
    // the distinct messages among them, in (origin step, sender) order, each with its receivers
    struct Msg { uint64_t origin; uint32_t sender, slot, receivers; };
    std::vector<Msg> msgs;
    for (uint32_t r = 0; r < W && r < 32; ++r)
        for (const Due& d : due[r]) {
            auto it = std::find_if(msgs.begin(), msgs.end(), [&](const Msg& m) { return m.slot == d.slot; });
            if (it == msgs.end()) msgs.push_back(Msg{d.origin, d.sender, d.slot, 1u << r});
            else it->receivers |= 1u << r;
        }
    std::sort(msgs.begin(), msgs.end(), [](const Msg& a, const Msg& b) {
        return a.origin != b.origin ? a.origin < b.origin : a.sender < b.sender;
    });
    if (!grid_shape().fuse_apply || W > 32 || msgs.size() > (size_t)kMaxStepMessages || total < 2) {
        for (uint32_t r = 0; r < W; ++r) {
            const int rc = apply_due(ctx, r, due[r]);
            if (rc != TENSAIR_OK) return rc;
        }
        return TENSAIR_OK;
    }
    StepMessages f;
    f.count = (uint32_t)msgs.size();
    for (size_t i = 0; i < msgs.size(); ++i) {
        f.ids[i] = ctx->slot_ids(msgs[i].slot);
        f.delta[i] = ctx->slot_delta(msgs[i].slot);
        f.buckets[i] = ctx->slot_buckets(msgs[i].slot);
        f.receivers[i] = msgs[i].receivers;
    }
    TENSAIR_CUDA(ctx, launch_apply_step(ctx->L, f, W, ctx->tables, (size_t)2 * ctx->cfg.V * ctx->cv.stride, ctx->shape, K_APPLY_STEP));
    return TENSAIR_OK;
}

int tensair_drain(tensair_ctx* ctx, uint32_t* n_applied) {
    if (!ctx) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    uint32_t total = 0;
    for (uint32_t r = 0; r < ctx->cfg.W; ++r) {
        const std::vector<Due> due = ctx->sched->take_due(ctx->gid(r), 0, true);
        total += (uint32_t)due.size();
        const int rc = apply_due(ctx, r, due);
        if (rc != TENSAIR_OK) return rc;
    }
    // the replicas held by other processes drain there; only their bookkeeping is kept here
    for (uint32_t g = 0; g < ctx->world_W; ++g)
        if (g < ctx->first || g >= ctx->first + ctx->cfg.W) ctx->sched->take_due(g, 0, true);
    if (n_applied) *n_applied = total;
    return TENSAIR_OK;
}

int tensair_message_buffers(tensair_ctx* ctx, uint32_t sender, uint64_t batch_index, tensair_msg_view* out) {
    if (!ctx || !out || sender >= ctx->world_W || batch_index >= (1ull << 32)) return TENSAIR_EINVAL;
    const uint32_t slot = ctx->sched->slot_of(sender, batch_index);
    const bool local = sender >= ctx->first && sender < ctx->first + ctx->cfg.W;
    // a local message must be the one held; a remote one is about to be received, so its slot must be free
    if (local ? !ctx->sched->slot_holds(slot, batch_index) : ctx->sched->slot_busy(slot))
        return local ? TENSAIR_ENOTFOUND : TENSAIR_EPENDING;
    out->ids = ctx->slot_ids(slot);
    out->delta = ctx->slot_delta(slot);
    out->max_rows = ctx->cv.slot_rows;
    out->row_stride = ctx->cv.stride;
    out->ids_offset = (uint64_t)slot * ctx->cv.slot_bytes + ctx->cv.ids_off;
    out->delta_offset = (uint64_t)slot * ctx->cv.slot_bytes + ctx->cv.delta_off;
    out->header_offset = (uint64_t)slot * ctx->cv.slot_bytes;
    return TENSAIR_OK;
}

int tensair_message_rows(tensair_ctx* ctx, uint32_t replica, uint64_t batch_index, uint32_t* n_rows, uint32_t* n_in_rows) {
    if (!ctx || replica >= ctx->cfg.W) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    const uint32_t slot = ctx->sched->slot_of(ctx->gid(replica), batch_index);
    if (!ctx->sched->slot_holds(slot, batch_index)) return TENSAIR_ENOTFOUND;
    TENSAIR_CUDA(ctx, cudaMemcpyAsync(&ctx->stage->hdr, ctx->slot_hdr(slot), sizeof(MsgHeader), cudaMemcpyDeviceToHost, ctx->stream));
    const int st = collect(ctx);
    if (st != TENSAIR_OK) return st;
    if (n_rows) *n_rows = ctx->stage->hdr.n_rows;
    if (n_in_rows) *n_in_rows = ctx->stage->hdr.n_in_rows;
    return TENSAIR_OK;
}

int tensair_commit_message(tensair_ctx* ctx, uint32_t sender, uint64_t batch_index, uint32_t n_rows, uint32_t n_in_rows) {
    return tensair_commit_message_on(ctx, sender, batch_index, n_rows, n_in_rows, nullptr);
}

int tensair_commit_message_on(tensair_ctx* ctx, uint32_t sender, uint64_t batch_index, uint32_t n_rows, uint32_t n_in_rows,
                              void* stream) {
    if (!ctx || sender >= ctx->world_W || batch_index >= (1ull << 32) || n_in_rows > n_rows || n_rows > ctx->cv.slot_rows)
        return TENSAIR_EINVAL;
    if (sender >= ctx->first && sender < ctx->first + ctx->cfg.W) return TENSAIR_EINVAL;   // local messages file themselves
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    const int rc = ctx->sched->on_train(sender, batch_index);
    if (rc != TENSAIR_OK) return rc;
    const uint32_t slot = ctx->sched->slot_of(sender, batch_index);
    Launcher L = ctx->L;
    if (stream) L.stream = (cudaStream_t)stream;
    TENSAIR_CUDA(ctx, launch_index_received(L, ctx->slot_hdr(slot), ctx->slot_ids(slot), ctx->slot_buckets(slot),
                                            ctx->cfg.V, n_rows, n_in_rows));
    return TENSAIR_OK;
}

int tensair_shadow_apply(tensair_ctx* ctx, uint32_t receiver, uint64_t step, int drain, uint32_t* n_applied) {
    if (!ctx || receiver >= ctx->world_W) return TENSAIR_EINVAL;
    if (receiver >= ctx->first && receiver < ctx->first + ctx->cfg.W) return TENSAIR_EINVAL;   // that one is applied for real
    const std::vector<Due> due = ctx->sched->take_due(receiver, step, drain != 0);
    if (n_applied) *n_applied = (uint32_t)due.size();
    return TENSAIR_OK;
}

namespace {

constexpr uint64_t kStateMagic = 0x3154535249415354ull;   // "TSAIRST1"

// The configuration a saved state belongs to, field by field.
std::vector<uint64_t> state_header(const tensair_ctx* ctx) {
    const tensair_config& c = ctx->cfg;
    uint32_t lr_bits;
    std::memcpy(&lr_bits, &c.lr, 4);
    return {kStateMagic, c.V, c.d, c.window, c.k, c.batch, c.W, lr_bits, c.max_grad_buffer, c.max_delay, ctx->cv.stride,
            c.seed, c.reduction, ctx->world_W, ctx->first};
}

}  // namespace

int tensair_save_state(tensair_ctx* ctx, void* host_dst, uint64_t capacity, uint64_t* bytes) {
    if (!ctx || !bytes) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    const int st = collect(ctx);
    if (st != TENSAIR_OK) return st;
    const std::vector<uint64_t> head = state_header(ctx);
    std::vector<uint8_t> sched;
    ctx->sched->save(sched);
    const uint64_t V = ctx->cfg.V;
    const uint64_t need = head.size() * 8 + 8 + ctx->buffered.size() * 8 + V * 16 + 8 + sched.size();
    *bytes = need;
    if (!host_dst) return TENSAIR_OK;
    if (capacity < need) return TENSAIR_ENOMEM;
    uint8_t* out = static_cast<uint8_t*>(host_dst);
    auto put = [&out](uint64_t v) { std::memcpy(out, &v, 8); out += 8; };
    for (uint64_t v : head) put(v);
    put(ctx->buffered.size());
    for (uint32_t b : ctx->buffered) put(b);
    TENSAIR_CUDA(ctx, cudaMemcpy(out, ctx->at<uint64_t>(ctx->cv.counts), V * 8, cudaMemcpyDeviceToHost));
    out += V * 8;
    TENSAIR_CUDA(ctx, cudaMemcpy(out, ctx->at<uint2>(ctx->cv.alias_tab), V * 8, cudaMemcpyDeviceToHost));
    out += V * 8;
    put(sched.size());
    std::memcpy(out, sched.data(), sched.size());
    return TENSAIR_OK;
}

int tensair_load_state(tensair_ctx* ctx, const void* host_src, uint64_t bytes) {
    if (!ctx || !host_src) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    const std::vector<uint64_t> head = state_header(ctx);
    const uint64_t V = ctx->cfg.V;
    const uint64_t fixed = head.size() * 8 + 8 + ctx->buffered.size() * 8 + V * 16 + 8;
    if (bytes < fixed) return TENSAIR_EINVAL;
    const uint8_t* in = static_cast<const uint8_t*>(host_src);
    auto get = [&in]() { uint64_t v; std::memcpy(&v, in, 8); in += 8; return v; };
    for (uint64_t v : head)
        if (get() != v) { ctx->last_error = "the saved state belongs to another configuration"; return TENSAIR_EINVAL; }
    if (get() != ctx->buffered.size()) return TENSAIR_EINVAL;
    std::vector<uint32_t> buffered(ctx->buffered.size());
    for (uint32_t& b : buffered) {
        const uint64_t v = get();
        if (v >= ctx->cfg.max_grad_buffer) return TENSAIR_EINVAL;
        b = (uint32_t)v;
    }
    const uint8_t* counts = in;
    const uint8_t* alias = in + V * 8;
    in += V * 16;
    const uint64_t sched_bytes = get();
    if (sched_bytes != bytes - fixed) return TENSAIR_EINVAL;
    // the schedule checks its own blob and changes nothing unless all of it is sound
    if (!ctx->sched->load(in, sched_bytes)) { ctx->last_error = "the saved delivery schedule is damaged"; return TENSAIR_EINVAL; }
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    TENSAIR_CUDA(ctx, cudaMemcpy(ctx->at<uint64_t>(ctx->cv.counts), counts, V * 8, cudaMemcpyHostToDevice));
    TENSAIR_CUDA(ctx, cudaMemcpy(ctx->at<uint2>(ctx->cv.alias_tab), alias, V * 8, cudaMemcpyHostToDevice));
    ctx->buffered = buffered;
    ctx->have_last = false;
    return TENSAIR_OK;
}

int tensair_update_sampler(tensair_ctx* ctx) {
    if (!ctx) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    if (grid_shape().device_alias_build) {
        // Every batch prepared ahead so far has been waited for by the caller's stream (its forward kernel follows its
        // sampling), so the table may be rewritten here; the batches prepared from now on wait for this event.
        TENSAIR_CUDA(ctx, launch_alias_build(ctx->L, ctx->at<unsigned long long>(ctx->cv.counts), ctx->cfg.V,
                                             ctx->at<AliasState>(ctx->cv.alias_state), ctx->at<uint8_t>(ctx->cv.alias_work),
                                             ctx->at<uint2>(ctx->cv.alias_tab)));
        if (ctx->prep) {
            TENSAIR_CUDA(ctx, cudaEventRecord(ctx->ev_sampler, ctx->stream));
            ctx->sampler_rebuilt = true;
        }
        return TENSAIR_OK;
    }
    std::vector<uint64_t> counts(ctx->cfg.V);
    TENSAIR_CUDA(ctx, cudaMemcpyAsync(counts.data(), ctx->at<uint64_t>(ctx->cv.counts), (size_t)ctx->cfg.V * 8, cudaMemcpyDeviceToHost, ctx->stream));
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return upload_sampler(ctx, counts.data());
}

int tensair_read_loss_async(tensair_ctx* ctx, double* host_dst) {
    if (!ctx || !host_dst || !ctx->have_last) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    TENSAIR_CUDA(ctx, cudaMemcpyAsync(host_dst, ctx->at<double>(ctx->cv.loss), 8, cudaMemcpyDeviceToHost, ctx->stream));
    return TENSAIR_OK;
}

int tensair_sync(tensair_ctx* ctx) {
    if (!ctx) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    return collect(ctx);
}

int tensair_read_embeddings(tensair_ctx* ctx, uint32_t replica, int which, uint32_t row0, uint32_t nrows, float* host_dst) {
    if (!ctx) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    return copy_rows(ctx, replica, which, row0, nrows, host_dst, true);
}

int tensair_write_embeddings(tensair_ctx* ctx, uint32_t replica, int which, uint32_t row0, uint32_t nrows, const float* host_src) {
    if (!ctx) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    return copy_rows(ctx, replica, which, row0, nrows, const_cast<float*>(host_src), false);
}

int tensair_snapshot_rows(tensair_ctx* ctx, uint32_t replica, int which, uint32_t row0, uint32_t nrows, float* snap_dev) {
    if (!ctx || replica >= ctx->cfg.W || (which != 0 && which != 1) || (uint64_t)row0 + nrows > ctx->cfg.V ||
        (!snap_dev && nrows))
        return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    if (!nrows) return TENSAIR_OK;
    const tensair_config& c = ctx->cfg;
    const float* src = ctx->table_of(replica) + ((size_t)which * c.V + row0) * ctx->cv.stride;
    TENSAIR_CUDA(ctx, cudaMemcpy2DAsync(snap_dev, (size_t)c.d * 4, src, (size_t)ctx->cv.stride * 4, (size_t)c.d * 4, nrows,
                                        cudaMemcpyDeviceToDevice, ctx->stream));
    return TENSAIR_OK;
}

int tensair_cosine_difference(tensair_ctx* ctx, uint32_t replica, int which, uint32_t row0, uint32_t nrows,
                              const float* snap_dev, float* out_dev) {
    if (!ctx || replica >= ctx->cfg.W || (which != 0 && which != 1) || (uint64_t)row0 + nrows > ctx->cfg.V ||
        ((!snap_dev || !out_dev) && nrows))
        return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    const tensair_config& c = ctx->cfg;
    const float* rows = ctx->table_of(replica) + ((size_t)which * c.V + row0) * ctx->cv.stride;
    TENSAIR_CUDA(ctx, launch_cosine_difference(ctx->L, rows, snap_dev, out_dev, nrows, ctx->shape));
    return TENSAIR_OK;
}

int tensair_top_drifted(tensair_ctx* ctx, const float* diff_dev, uint32_t nrows, uint32_t k, uint32_t* ids_dev,
                        float* vals_dev, uint32_t* n_out) {
    if (!ctx || k > kTopkMax) return TENSAIR_EINVAL;
    const uint32_t m = k < nrows ? k : nrows;
    if (m && (!diff_dev || !ids_dev || !vals_dev)) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    TENSAIR_CUDA(ctx, launch_top_drifted(ctx->L, diff_dev, nrows, m, ctx->at<TopkState>(ctx->cv.topk), ids_dev, vals_dev));
    if (n_out) *n_out = m;
    return TENSAIR_OK;
}

int tensair_read_negatives(tensair_ctx* ctx, uint32_t* host_neg, uint32_t* n_pairs) {
    if (!ctx || !ctx->have_last) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    if (n_pairs) *n_pairs = ctx->last_pairs;
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (host_neg && ctx->last_pairs) {
        const uint32_t k = ctx->cfg.k;
        // rows are stored per pair as [positive, k negatives]
        TENSAIR_CUDA(ctx, cudaMemcpy2D(host_neg, (size_t)k * 4, (ctx->last_rows ? ctx->last_rows : ctx->at<uint32_t>(ctx->cv.rows)) + 1, (size_t)(k + 1) * 4,
                                       (size_t)k * 4, ctx->last_pairs, cudaMemcpyDeviceToHost));
    }
    return TENSAIR_OK;
}

int tensair_read_scalars(tensair_ctx* ctx, double* host_g) {
    if (!ctx || !ctx->have_last || !host_g) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    const size_t n = (size_t)ctx->last_pairs * (ctx->cfg.k + 1);
    if (n) TENSAIR_CUDA(ctx, cudaMemcpy2D(host_g, 8, ctx->at<Rec>(ctx->cv.rec), sizeof(Rec), 8, n, cudaMemcpyDeviceToHost));
    return TENSAIR_OK;
}

int tensair_read_message(tensair_ctx* ctx, uint32_t replica, uint64_t batch_index, uint32_t* n_rows,
                         uint32_t* host_ids, float* host_delta) {
    if (!ctx || replica >= ctx->world_W) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    const uint32_t slot = ctx->sched->slot_of(replica, batch_index);
    if (!ctx->sched->slot_holds(slot, batch_index)) return TENSAIR_ENOTFOUND;
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    MsgHeader h;
    TENSAIR_CUDA(ctx, cudaMemcpy(&h, ctx->slot_hdr(slot), sizeof(h), cudaMemcpyDeviceToHost));
    if (n_rows) *n_rows = h.n_rows;
    if (host_ids && h.n_rows) TENSAIR_CUDA(ctx, cudaMemcpy(host_ids, ctx->slot_ids(slot), (size_t)h.n_rows * 4, cudaMemcpyDeviceToHost));
    if (host_delta && h.n_rows)
        TENSAIR_CUDA(ctx, cudaMemcpy2D(host_delta, (size_t)ctx->cfg.d * 4, ctx->slot_delta(slot), (size_t)ctx->cv.stride * 4,
                                       (size_t)ctx->cfg.d * 4, h.n_rows, cudaMemcpyDeviceToHost));
    return TENSAIR_OK;
}

int tensair_read_sampler(tensair_ctx* ctx, uint32_t* thresh, uint32_t* alias, uint64_t* counts) {
    if (!ctx) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    const uint32_t V = ctx->cfg.V;
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (thresh || alias) {
        std::vector<uint2> packed(V);
        TENSAIR_CUDA(ctx, cudaMemcpy(packed.data(), ctx->at<uint2>(ctx->cv.alias_tab), (size_t)V * 8, cudaMemcpyDeviceToHost));
        for (uint32_t i = 0; i < V; ++i) {
            if (thresh) thresh[i] = packed[i].x;
            if (alias) alias[i] = packed[i].y;
        }
    }
    if (counts) TENSAIR_CUDA(ctx, cudaMemcpy(counts, ctx->at<uint64_t>(ctx->cv.counts), (size_t)V * 8, cudaMemcpyDeviceToHost));
    return TENSAIR_OK;
}

int tensair_read_delivery_log(tensair_ctx* ctx, uint32_t replica, uint64_t max_records, tensair_delivery* out, uint64_t* n) {
    if (!ctx || replica >= ctx->cfg.W) return TENSAIR_EINVAL;
    const std::vector<tensair_delivery>& lg = ctx->sched->log(ctx->gid(replica));
    if (n) *n = lg.size();
    for (uint64_t i = 0; i < lg.size() && i < max_records && out; ++i) out[i] = lg[i];
    return TENSAIR_OK;
}

int tensair_pending(tensair_ctx* ctx, uint32_t replica, uint64_t* n) {
    if (!ctx || !n || replica >= ctx->cfg.W) return TENSAIR_EINVAL;
    *n = ctx->sched->pending(ctx->gid(replica));
    return TENSAIR_OK;
}

uint64_t tensair_kernel_launches(const tensair_ctx* ctx) { return ctx ? ctx->launches : 0; }

int tensair_tune(const char* name, int value) {
    if (!name) return TENSAIR_EINVAL;
    static int rows = 0, blocks = 0;
    if (!std::strcmp(name, "forward_rows")) rows = value;
    else if (!std::strcmp(name, "forward_blocks_per_sm")) blocks = value;
    else if (!std::strcmp(name, "fused_blocks_per_sm") && value > 0) { grid_shape().fused_blocks_per_sm = value; return TENSAIR_OK; }
    else if (!std::strcmp(name, "fuse_apply")) { grid_shape().fuse_apply = value; return TENSAIR_OK; }
    else if (!std::strcmp(name, "overlap_sort")) { grid_shape().overlap_sort = value; return TENSAIR_OK; }
    else if (!std::strcmp(name, "early_prepare") && value >= 0 && value <= 2) { grid_shape().early_prepare = value; return TENSAIR_OK; }
    else if (!std::strcmp(name, "early_prepare_max_items") && value >= 0) { grid_shape().early_prepare_max_items = value; return TENSAIR_OK; }
    else if (!std::strcmp(name, "overlap_long_rows")) { grid_shape().overlap_long_rows = value; return TENSAIR_OK; }
    else if (!std::strcmp(name, "device_alias_build")) { grid_shape().device_alias_build = value; return TENSAIR_OK; }
    else if (!std::strcmp(name, "reduce_blocks_per_sm") && value > 0) { grid_shape().reduce_blocks_per_sm = value; return TENSAIR_OK; }
    else if (!std::strcmp(name, "apply_blocks_per_sm") && value > 0) { grid_shape().apply_blocks_per_sm = value; return TENSAIR_OK; }
    else return TENSAIR_EINVAL;
    set_forward_shape(rows, blocks);
    return TENSAIR_OK;
}

int tensair_profile(tensair_ctx* ctx, int enable) {
    if (!ctx) return TENSAIR_EINVAL;
    ctx->prof.on = enable != 0;
    return TENSAIR_OK;
}

int tensair_profile_read(tensair_ctx* ctx, uint32_t max_kinds, tensair_kernel_time* out, uint32_t* n_kinds) {
    if (!ctx) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    double total[K_KINDS] = {0};
    uint64_t count[K_KINDS] = {0};
    for (const Profiler::Span& sp : ctx->prof.spans) {
        float ms = 0.0f;
        TENSAIR_CUDA(ctx, cudaEventElapsedTime(&ms, sp.start, sp.stop));
        total[sp.kind] += ms;
        ++count[sp.kind];
        ctx->prof.spare.push_back(sp.start);
        ctx->prof.spare.push_back(sp.stop);
    }
    ctx->prof.spans.clear();
    if (n_kinds) *n_kinds = K_KINDS;
    for (uint32_t i = 0; i < K_KINDS && i < max_kinds && out; ++i) {
        std::memset(&out[i], 0, sizeof(out[i]));
        std::snprintf(out[i].name, sizeof(out[i].name), "%s", kernel_name((int)i));
        out[i].launches = count[i];
        out[i].total_ms = total[i];
    }
    return TENSAIR_OK;
}

const char* tensair_strerror(int code) {
    switch (code) {
        case TENSAIR_OK: return "ok";
        case TENSAIR_EINVAL: return "invalid argument or unsupported configuration";
        case TENSAIR_ENOMEM: return "a caller-provided buffer is too small";
        case TENSAIR_ECUDA: return "a CUDA call failed";
        case TENSAIR_EBADTOKEN: return "token id outside [0,V)";
        case TENSAIR_EPENDING: return "message slot still has undelivered recipients";
        case TENSAIR_ENOTFOUND: return "message no longer held";
        case TENSAIR_ETIMEOUT: return "a bounded wait inside a kernel ran out";
        case TENSAIR_EBOUNDS: return "an index checked on the device was outside its array";
        default: return "unknown error";
    }
}

const char* tensair_last_error(const tensair_ctx* ctx) { return ctx ? ctx->last_error.c_str() : ""; }

int tensair_error_of_flags(uint32_t flags) { return error_of_flags(flags, nullptr); }

int tensair_checked_build(void) {
#ifdef TENSAIR_BOUNDS
    return 1;
#else
    return 0;
#endif
}

int tensair_raise_error_flags(tensair_ctx* ctx, uint32_t flags) {
    if (!ctx) return TENSAIR_EINVAL;
    DeviceGuard guard(ctx->cfg.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    // the word is sticky: OR the bits in by reading it back first (a test hook, so the round trip does not matter)
    TENSAIR_CUDA(ctx, cudaMemcpyAsync(&ctx->stage->err, ctx->at<uint32_t>(ctx->cv.err), 4, cudaMemcpyDeviceToHost, ctx->stream));
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    ctx->stage->err |= flags;
    TENSAIR_CUDA(ctx, cudaMemcpyAsync(ctx->at<uint32_t>(ctx->cv.err), &ctx->stage->err, 4, cudaMemcpyHostToDevice, ctx->stream));
    TENSAIR_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return TENSAIR_OK;
}

int tensair_build_alias_host(const uint64_t* counts, uint32_t V, uint32_t* thresh, uint32_t* alias) {
    if (!V || !thresh || !alias) return TENSAIR_EINVAL;
    if (counts)
        for (uint32_t i = 0; i < V; ++i) if (counts[i] < 1) return TENSAIR_EINVAL;
    build_alias_host(counts, V, thresh, alias);
    return TENSAIR_OK;
}

}  // extern "C"
