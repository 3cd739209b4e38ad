// tensair_train_batch_static: the mini-batch step with its per-batch working memory inside the library.
//
// Some callers hold a context but may not allocate device memory at the moment they train: code that
// runs between the allocation phases of a host application with a fixed memory plan, a plug-in that is
// handed tables and a message pool by its host and nothing else, a service thread that must not call
// into the allocator.  For them this entry point takes the sort buffers, segment lists and partial
// sums of one batch from a fixed array that is part of the library image instead of from a
// caller-sized scratch buffer.  Inputs (tokens, the context with its tables and sampler state) and
// outputs (tables, message slot, loss) are the caller's as in tensair_train_batch.
//
// The array is `static __device__`: every GPU that loads the library reserves kStaticScratchBytes of
// device memory for it until the process exits, whether or not this entry point is ever called.  In
// host code the array's name is only a handle; the device address is obtained once per device with
// cudaGetSymbolAddress while that device is current, on the first call for that device.
#include <cstdio>
#include <cstring>
#include <mutex>

#include "context.h"

using namespace tensair;

namespace {

constexpr size_t kStaticScratchBytes = 32u << 20;   // 32 MiB per GPU
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

unsigned char* g_scratch_address[kMaxDevices];      // device address of the array, per device ordinal
bool g_scratch_known[kMaxDevices];
std::mutex g_scratch_lock;                          // first calls may come from several host threads

// Byte offsets of the per-batch working buffers inside the array (same sizes as the context's own scratch).
struct StaticCarve {
    uint64_t long_counters, items_a, items_b, terms, gin_pos, loss_pos, hist, tile_counts, seg_start, long_rows,
        chunk_items, partials, total;
};

void carve_static(const tensair_config& c, const Carve& cv, StaticCarve& k) {
    uint64_t off = 0;
    auto take = [&off](uint64_t bytes) { const uint64_t at = off; off = round_up(off + bytes, 256); return at; };
    k.long_counters = take(16);
    k.items_a = take((uint64_t)cv.max_items * 8);
    k.items_b = take((uint64_t)cv.max_items * 8);
    k.terms = take((uint64_t)cv.max_items * sizeof(Rec));
    k.gin_pos = take((uint64_t)2 * c.batch * cv.stride * 8);
    k.loss_pos = take((uint64_t)2 * c.batch * 8);
    k.hist = take((uint64_t)sort_hist_words(cv.max_items) * 4);
    k.tile_counts = take((uint64_t)(heads_tiles(cv.max_items) + 1) * 4);
    k.seg_start = take((uint64_t)(cv.max_rows + 2) * 4);
    k.long_rows = take((uint64_t)cv.max_long * sizeof(LongRow));
    k.chunk_items = take((uint64_t)cv.max_chunks * sizeof(ChunkItem));
    k.partials = take((uint64_t)cv.max_chunks * cv.stride * 8);
    k.total = off;
}

}  // namespace

extern "C" int tensair_train_batch_static(tensair_ctx* ctx, uint32_t replica, const int32_t* tokens_dev,
                                          uint32_t n_tokens, uint64_t batch_index, double* loss_out,
                                          tensair_msg_info* info) {
    if (!ctx || replica >= ctx->cfg.W || n_tokens > ctx->cfg.batch || (n_tokens && !tokens_dev) ||
        batch_index >= (1ull << 32))
        return TENSAIR_EINVAL;
    const tensair_config& c = ctx->cfg;
    const Carve& cv = ctx->cv;
    if (c.device < 0 || c.device >= kMaxDevices) return TENSAIR_EINVAL;
    if (c.max_grad_buffer != 1) return TENSAIR_EINVAL;   // buffered gradients are only handled by tensair_train_batch
    StaticCarve sc;
    carve_static(c, cv, sc);
    if (sc.total > kStaticScratchBytes) {
        char msg[200];
        std::snprintf(msg, sizeof(msg),
                      "tensair_train_batch_static: this configuration needs %llu bytes of per-batch scratch, "
                      "the built-in array holds %llu",
                      (unsigned long long)sc.total, (unsigned long long)kStaticScratchBytes);
        ctx->last_error = msg;
        return TENSAIR_ENOMEM;
    }
    DeviceGuard guard(c.device);
    if (!guard.ok) return TENSAIR_ECUDA;
    unsigned char* ws = nullptr;
    {
        std::lock_guard<std::mutex> hold(g_scratch_lock);
        if (!g_scratch_known[c.device]) {
            // set-up, once per device, with that device current: the symbol is not a device pointer in host code
            unsigned char* ptr = nullptr;
            TENSAIR_CUDA(ctx, cudaGetSymbolAddress((void**)&ptr, g_static_scratch));
            g_scratch_address[c.device] = ptr;
            g_scratch_known[c.device] = true;
        }
        ws = g_scratch_address[c.device];
    }
    auto in_ws = [ws](uint64_t off) { return ws + off; };

    const uint32_t me = ctx->gid(replica);   // the replica's id among all replicas of the job
    const int rc = ctx->sched->on_train(me, batch_index);
    if (rc != TENSAIR_OK) return rc;
    const uint32_t slot = ctx->sched->slot_of(me, batch_index);
    const uint32_t pairs = n_tokens >= 2 ? pair_count(n_tokens, c.window) : 0;
    const uint32_t n_items = pairs ? 2 * n_tokens + pairs * (c.k + 1) : 0;
    uint32_t* err = ctx->at<uint32_t>(cv.err);
    float* table = ctx->table_of(replica);
    MsgHeader* hdr = ctx->slot_hdr(slot);
    const double scale = c.reduction == TENSAIR_MEAN && pairs ? (double)c.lr / (double)pairs : (double)c.lr;
    item_t* items_a = reinterpret_cast<item_t*>(in_ws(sc.items_a));
    item_t* items_b = reinterpret_cast<item_t*>(in_ws(sc.items_b));
    Rec* terms = reinterpret_cast<Rec*>(in_ws(sc.terms));
    double* gin_pos = reinterpret_cast<double*>(in_ws(sc.gin_pos));
    double* loss_pos = reinterpret_cast<double*>(in_ws(sc.loss_pos));
    uint32_t* long_counters = reinterpret_cast<uint32_t*>(in_ws(sc.long_counters));

    // the array keeps what the previous call left: the list counters must start at zero
    TENSAIR_CUDA(ctx, cudaMemsetAsync(long_counters, 0, 16, ctx->stream));
    TENSAIR_CUDA(ctx, launch_validate(ctx->L, tokens_dev, n_tokens, c.V, err, nullptr, nullptr, nullptr, ctx->world_W, me, c.seed));
    TENSAIR_CUDA(ctx, launch_prepare(ctx->L, tokens_dev, n_tokens, ctx->shape, me, (uint32_t)batch_index, c.seed,
                                     ctx->at<uint2>(cv.alias_tab), ctx->at<uint32_t>(cv.rows), items_a,
                                     ctx->at<unsigned long long>(cv.counts), err, nullptr, false, true));
    if (n_items) {
        TENSAIR_CUDA(ctx, launch_forward(ctx->L, tokens_dev, n_tokens, ctx->shape, table, ctx->at<uint32_t>(cv.rows),
                                         ctx->at<Rec>(cv.rec), gin_pos, loss_pos, err, nullptr, nullptr));
        item_t* sorted = nullptr;
        TENSAIR_CUDA(ctx, launch_sort(ctx->L, items_a, items_b, n_items, bits_for(2 * c.V),
                                      reinterpret_cast<uint32_t*>(in_ws(sc.hist)), &sorted));
        TENSAIR_CUDA(ctx, launch_heads(ctx->L, sorted, n_items, c.V, reinterpret_cast<uint32_t*>(in_ws(sc.tile_counts)), hdr,
                                       ctx->slot_ids(slot), reinterpret_cast<uint32_t*>(in_ws(sc.seg_start)),
                                       long_counters, ctx->at<Rec>(cv.rec), terms, err,
                                       reinterpret_cast<LongRow*>(in_ws(sc.long_rows)),
                                       reinterpret_cast<ChunkItem*>(in_ws(sc.chunk_items)), nullptr, 0, nullptr, nullptr));
        TENSAIR_CUDA(ctx, launch_reduce_rows(ctx->L, terms, hdr, ctx->slot_ids(slot),
                                             reinterpret_cast<uint32_t*>(in_ws(sc.seg_start)), gin_pos, table,
                                             ctx->slot_delta(slot), ctx->shape, scale));
        TENSAIR_CUDA(ctx, launch_reduce_long_rows(ctx->L, terms, ctx->slot_ids(slot),
                                                  reinterpret_cast<uint32_t*>(in_ws(sc.seg_start)), gin_pos, table,
                                                  ctx->slot_delta(slot), ctx->shape, scale, long_counters,
                                                  reinterpret_cast<LongRow*>(in_ws(sc.long_rows)),
                                                  reinterpret_cast<ChunkItem*>(in_ws(sc.chunk_items)),
                                                  reinterpret_cast<double*>(in_ws(sc.partials))));
        TENSAIR_CUDA(ctx, launch_apply_rows(ctx->L, hdr, ctx->slot_ids(slot), ctx->slot_delta(slot), table, ctx->shape, 1));
    } else {
        TENSAIR_CUDA(ctx, cudaMemsetAsync(hdr, 0, sizeof(MsgHeader), ctx->stream));
    }
    TENSAIR_CUDA(ctx, launch_bucket_index(ctx->L, hdr, ctx->slot_ids(slot), ctx->slot_buckets(slot), c.V));
    TENSAIR_CUDA(ctx, launch_loss_sum(ctx->L, loss_pos, n_tokens, ctx->at<double>(cv.loss), err, nullptr));
    ctx->last_n = n_tokens;
    ctx->last_pairs = pairs;
    ctx->have_last = true;
    ctx->last_rows = ctx->at<uint32_t>(cv.rows);      // where this call left its row ids (parity tap)
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
