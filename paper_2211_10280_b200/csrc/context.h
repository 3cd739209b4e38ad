// The context behind the C ABI and the helpers every entry point shares.
#pragma once
#include <stdint.h>

#include <string>
#include <vector>

#include "../../include/tensair.h"
#include "kernels.h"
#include "schedule.h"

namespace tensair {

inline uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

// Offsets (bytes) of everything the library keeps in the caller's scratch buffer.
struct Carve {
    uint64_t err, loss, long_counters, counts, alias_tab, tok, rows, items_a, items_b, rec, terms, gin_pos, loss_pos, hist,
        tile_counts, seg_start, long_rows, chunk_items, partials, merge_counts, topk, owner, owned, n_owned, alias_state, alias_work, total;
    // buffer sets of the batches prepared ahead of their turn (tokens, row ids, sort buffers, histograms, error word)
    uint64_t set_base, set_bytes, set_tok, set_rows, set_items_a, set_items_b, set_hist, set_err;
    uint64_t slot_bytes, bucket_off, ids_off, delta_off;
    uint32_t stride, max_pairs, max_contrib, max_items, max_long, max_chunks;
    uint32_t max_rows;    // most rows the message of ONE batch can have (bounds the per-batch lists)
    uint32_t slot_rows;   // rows a message slot holds: max_rows, or the union of maxGradBuffer buffered messages
};

inline uint32_t bits_for(uint32_t x) {   // bits needed to represent x
    uint32_t b = 0;
    while (x) { ++b; x >>= 1; }
    return b ? b : 1;
}

}  // namespace tensair

struct tensair_ctx {
    tensair_config cfg;
    tensair::Carve cv;
    tensair::Shape shape;
    cudaStream_t stream;
    // internal second stream: the sort of a batch's contributions runs there, beside the forward kernel
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    tensair::Launcher L_side;
    tensair::Launcher L;
    // Third stream: the sampling and the sort of a batch need only its tokens and the sampler table, so they run here,
    // ahead of the batch's turn on the caller's stream (beside the previous batches' kernels or the message application).
    static constexpr int kPrepSets = 4;
    cudaStream_t prep = nullptr;
    tensair::Launcher L_prep;
    cudaEvent_t ev_call = nullptr, ev_sampler = nullptr;
    cudaEvent_t ev_prepared[kPrepSets] = {}, ev_sorted[kPrepSets] = {}, ev_set_free[kPrepSets] = {};
    bool set_used[kPrepSets] = {};
    bool sampler_rebuilt = false;    // ev_sampler has been recorded at least once
    int next_set = 0, last_prepared = -1;
    const uint32_t* last_rows = nullptr;   // row ids of the most recent batch (parity tap)
    uint64_t launches = 0;
    tensair::Profiler prof;
    float* tables;
    uint8_t* pool;
    uint8_t* scratch;
    tensair::Schedule* sched = nullptr;
    // Replicas of the whole job and the global id of local replica 0.  One process holding every replica has
    // world_W == cfg.W and first == 0; in a sharded job cfg.W counts the replicas whose tables live here.
    uint32_t world_W = 0, first = 0;
    uint32_t gid(uint32_t local) const { return first + local; }
    std::vector<uint32_t> buffered;        // per replica: gradient messages computed and not yet sent (maxGradBuffer > 1)
    uint32_t last_n = 0, last_pairs = 0;
    bool have_last = false;
    std::string last_error;
    // pinned host staging for small read-backs
    struct Staging { tensair::MsgHeader hdr; double loss; uint32_t err; } *stage = nullptr;

    template <class T> T* at(uint64_t off) const { return reinterpret_cast<T*>(scratch + off); }
    template <class T> T* in_set(int set, uint64_t off) const {
        return reinterpret_cast<T*>(scratch + cv.set_base + (uint64_t)set * cv.set_bytes + off);
    }
    float* table_of(uint32_t replica) const { return tables + (size_t)replica * 2 * cfg.V * cv.stride; }
    uint8_t* slot_ptr(uint32_t slot) const { return pool + (size_t)slot * cv.slot_bytes; }
    tensair::MsgHeader* slot_hdr(uint32_t slot) const { return reinterpret_cast<tensair::MsgHeader*>(slot_ptr(slot)); }
    uint32_t* slot_buckets(uint32_t slot) const { return reinterpret_cast<uint32_t*>(slot_ptr(slot) + cv.bucket_off); }
    uint32_t* slot_ids(uint32_t slot) const { return reinterpret_cast<uint32_t*>(slot_ptr(slot) + cv.ids_off); }
    float* slot_delta(uint32_t slot) const { return reinterpret_cast<float*>(slot_ptr(slot) + cv.delta_off); }
};

namespace tensair {

// Records the CUDA error text on the context and returns TENSAIR_ECUDA.
int fail(tensair_ctx* ctx, cudaError_t e, const char* what);
// Waits for the stream, then reads and clears the device error word.
int collect(tensair_ctx* ctx);
// The code and text that a value of the device error word stands for.
int error_of_flags(uint32_t flags, std::string* text);

#define TENSAIR_CUDA(ctx, call)                                    \
    do {                                                           \
        const cudaError_t e_ = (call);                             \
        if (e_ != cudaSuccess) return tensair::fail((ctx), e_, #call);      \
    } while (0)

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace tensair
