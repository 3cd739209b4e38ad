// Host-side launchers of the kernels; each enqueues on L.stream and returns the launch status.
#pragma once
#include <vector>

#include "common.cuh"

namespace tensair {

enum KernelKind {
    K_VALIDATE, K_PREPARE, K_SORT_HIST, K_SORT_SCAN, K_SORT_SCATTER, K_FORWARD, K_LOSS_SUM, K_HEADS_COUNT,
    K_HEADS_WRITE, K_REDUCE_ROWS, K_REDUCE_CHUNKS, K_REDUCE_LONG, K_APPLY_INPUT_ROWS,
    K_APPLY_MESSAGE, K_INIT_TABLE, K_BUCKET_INDEX, K_APPLY_FUSED, K_COSINE, K_MERGE, K_TOPK, K_ALIAS_BUILD,
    K_APPLY_STEP, K_KINDS
};
inline const char* kernel_name(int kind) {
    static const char* const names[K_KINDS] = {
        "validate", "prepare", "sort_hist", "sort_scan", "sort_scatter", "forward", "loss_sum", "heads_count",
        "heads_write", "reduce_rows", "reduce_chunks", "reduce_long", "apply_input_rows",
        "apply_message", "init_table", "bucket_index", "apply_fused", "cosine_difference", "merge", "top_drifted", "alias_build",
        "apply_step"};
    return kind >= 0 && kind < K_KINDS ? names[kind] : "?";
}

// Optional per-launch timing: a pair of CUDA events around every kernel launch while `on` is set.
struct Profiler {
    struct Span { int kind; cudaEvent_t start, stop; };
    bool on = false;
    std::vector<Span> spans;
    std::vector<cudaEvent_t> spare;
    cudaEvent_t take() {
        cudaEvent_t e = nullptr;
        if (!spare.empty()) { e = spare.back(); spare.pop_back(); }
        else cudaEventCreate(&e);
        return e;
    }
};

struct Launcher {
    cudaStream_t stream;
    uint64_t* launches;   // incremented once per kernel launch
    int sms;              // multiprocessors of the device
    Profiler* prof;       // nullable
    int device = 0;       // ordinal of the device the stream belongs to
    Limits lim = {};      // array bounds handed to the kernels (used by the checked build only)
};
constexpr int kMaxDevices = 64;   // per-device launch state (function attributes, symbol addresses) is kept up to here

// Blocks per multiprocessor of the grid-stride kernels (row sums, message apply).  More blocks than
// are resident at once let the hardware scheduler even out rows of unequal cost.
struct GridShape {
    int fuse_apply = 1;              // apply the messages due for a receiver in one pass over its table
    int overlap_sort = 1;            // run the radix sort on a second stream while the forward kernel runs
    int early_prepare = 1;           // sample and sort a batch on a third stream ahead of its turn: 0 never, 1 when the tokens come from host memory, 2 also for device tokens (the caller vouches that they are complete when the call is made)
    int overlap_long_rows = 1;       // sum the long rows (and index the message, sum the loss) on it while the short rows are summed
    int device_alias_build = 1;      // rebuild the sampler's alias table on the device (0: on the host, with a synchronisation)
    int early_prepare_max_items = 1 << 20;   // ... for batches of at most this many sort items (larger ones gain nothing from it)
    int reduce_blocks_per_sm = 64;
    int apply_blocks_per_sm = 64;
    int fused_blocks_per_sm = 256;
};
GridShape& grid_shape();

// Counts one kernel launch and, when profiling, brackets it with events: construct right before the
// launch, let it go out of scope right after.
struct Timed {
    const Launcher& L;
    cudaEvent_t stop = nullptr;
    Timed(const Launcher& l, int kind) : L(l) {
        ++*L.launches;
        if (L.prof && L.prof->on) {
            cudaEvent_t start = L.prof->take();
            stop = L.prof->take();
            cudaEventRecord(start, L.stream);
            L.prof->spans.push_back(Profiler::Span{kind, start, stop});
        }
    }
    ~Timed() { if (stop) cudaEventRecord(stop, L.stream); }
};

// sampler.cu
cudaError_t launch_validate(const Launcher& L, const int32_t* tok, uint32_t n, uint32_t V, uint32_t* err, uint8_t* owner,
                            uint32_t* owned, uint32_t* n_owned, uint32_t W, uint32_t replica, uint64_t seed);
cudaError_t launch_prepare(const Launcher& L, const int32_t* tok, uint32_t n, const Shape& s, uint32_t replica,
                           uint32_t batch_lo, uint64_t seed, const uint2* alias_tab, uint32_t* rows,
                           item_t* items, unsigned long long* counts, uint32_t* err, const uint8_t* owner, bool check,
                           bool count);
cudaError_t launch_init_input_table(const Launcher& L, float* table, const Shape& s, uint64_t seed);
void build_alias_host(const uint64_t* counts, uint32_t V, uint32_t* thresh, uint32_t* alias);
int alias_mass_bits(uint32_t V);

// alias_build.cu: the same table built on the device from the running counts
struct AliasState {
    unsigned long long heaviest_bits;   // bit pattern of the largest weight
    unsigned long long sum, top;        // sum and maximum of the integer masses
    unsigned long long first_top;       // smallest index holding the maximum
    uint32_t lights, pad;               // entries lighter than a bucket's capacity
};
size_t alias_work_bytes(uint32_t V);
cudaError_t launch_alias_build(const Launcher& L, const unsigned long long* counts, uint32_t V, AliasState* st,
                               uint8_t* work, uint2* table);

// radix_sort.cu
// Stable least-significant-digit radix sort of `n` items by the low `key_bits` bits of their keys.
// `a` holds the input; `b` and `hist` are scratch.  *sorted receives whichever of a / b holds the result.
cudaError_t launch_sort(const Launcher& L, item_t* a, item_t* b, uint32_t n, uint32_t key_bits, uint32_t* hist,
                        item_t** sorted);
uint32_t sort_tiles(uint32_t n);
uint32_t sort_hist_words(uint32_t n);

// forward.cu
cudaError_t launch_forward(const Launcher& L, const int32_t* tok, uint32_t n, const Shape& s, const float* table,
                           const uint32_t* rows, Rec* rec, double* gin_pos, double* loss_pos, uint32_t* err,
                           const uint32_t* owned, const uint32_t* n_owned, const uint32_t* batch_err = nullptr,
                           bool sort_runs_beside = true);
void set_forward_shape(int rows, int blocks_per_sm);
cudaError_t launch_loss_sum(const Launcher& L, const double* loss_pos, uint32_t n, double* loss, const uint32_t* err,
                            const uint8_t* owner);

// message.cu
uint32_t heads_tiles(uint32_t n_items);
// tok / counts / owner: when counts is given, the batch's n tokens are added to the running unigram counts here
// (the first kernel that runs once the whole batch is known to be valid); nullptr = they were counted already.
// long_counters: 4 words (long rows, chunks, and the ticket that picks the block that scans the tile counts).
cudaError_t launch_heads(const Launcher& L, const item_t* sorted, uint32_t n_items, uint32_t V, uint32_t* tile_counts,
                         MsgHeader* hdr, uint32_t* ids, uint32_t* seg_start, uint32_t* long_counters,
                         const Rec* rec, Rec* terms, const uint32_t* err, LongRow* long_rows, ChunkItem* chunk_items,
                         const int32_t* tok, uint32_t n, unsigned long long* counts, const uint8_t* owner);
cudaError_t launch_reduce_rows(const Launcher& L, const Rec* terms, const MsgHeader* hdr, const uint32_t* ids,
                               const uint32_t* seg_start, const double* gin_pos, float* table, float* delta,
                               const Shape& s, double scale);
cudaError_t launch_reduce_long_rows(const Launcher& L, const Rec* terms, const uint32_t* ids, const uint32_t* seg_start,
                                    const double* gin_pos, float* table, float* delta, const Shape& s, double scale,
                                    const uint32_t* long_counters, const LongRow* long_rows,
                                    const ChunkItem* chunk_items, double* partials);

// apply.cu
cudaError_t launch_apply(const Launcher& L, const MsgHeader* hdr, const uint32_t* ids, const float* delta,
                         float* table, const Shape& s);
// Everything due in one step, for all receivers of the context, in one pass: the messages in (origin step,
// sender) order, each with the set of receivers it is due for.  Every (row, receiver) pair is fetched once,
// receives the deltas of its messages in message order and is stored once.
constexpr int kMaxStepMessages = 32;
struct StepMessages {
    uint32_t count;
    const uint32_t* ids[kMaxStepMessages];
    const float* delta[kMaxStepMessages];
    const uint32_t* buckets[kMaxStepMessages];
    uint32_t receivers[kMaxStepMessages];   // bit r set: add to the table of local replica r
};
// kind: K_APPLY_STEP, or K_APPLY_FUSED when the pass serves one receiver (tables = that receiver's table).
cudaError_t launch_apply_step(const Launcher& L, const StepMessages& f, uint32_t n_receivers, float* tables,
                              size_t replica_floats, const Shape& s, int kind);
// merge.cu: the sum of up to kMaxMerge buffered messages (each with its bucket index) into one message.
constexpr int kMaxMerge = 8;
struct MergeInputs {
    uint32_t count;
    const uint32_t* ids[kMaxMerge];
    const float* delta[kMaxMerge];
    const uint32_t* buckets[kMaxMerge];
};
// capacity: rows the output slot holds; a union with more rows raises kErrOverflow and is cut there.
cudaError_t launch_merge(const Launcher& L, const MergeInputs& in, MsgHeader* hdr, uint32_t* bucket_start, uint32_t* ids,
                         float* delta, uint32_t* counts, const Shape& s, uint32_t capacity, uint32_t* err);
// out[r] = 1 - cos(table row r, snapshot row r) for nrows rows; rows of `rows` are strided, of `snap` dense.
// Working state of the most-drifted-rows selection, in the context's scratch.
constexpr uint32_t kTopkMax = 4096;
struct TopkState {
    uint64_t prefix;        // leading bytes of the k-th largest rank key found so far
    uint32_t remaining;     // rank of that key among the keys sharing the prefix
    uint32_t n_out;
    uint32_t hist[256];
    uint64_t keys[kTopkMax];
};
cudaError_t launch_top_drifted(const Launcher& L, const float* diff, uint32_t n, uint32_t k, TopkState* st,
                               uint32_t* ids, float* vals);
cudaError_t launch_cosine_difference(const Launcher& L, const float* rows, const float* snap, float* out, uint32_t nrows,
                                     const Shape& s);
// bucket_start[b] = first row of the message with id >= b << kBucketShift, for b in [0, bucket_count(V)].
// loss != nullptr: the same launch also adds up the batch's loss from the 2n per-half-position losses (see
// launch_loss_sum, which does that on its own).
cudaError_t launch_bucket_index(const Launcher& L, const MsgHeader* hdr, const uint32_t* ids, uint32_t* bucket_start,
                                uint32_t V, const double* loss_pos = nullptr, uint32_t n = 0, double* loss = nullptr,
                                const uint32_t* err = nullptr, const uint8_t* owner = nullptr);
// The index of a message received from another process; also writes the slot's header from the given counts.
cudaError_t launch_index_received(const Launcher& L, MsgHeader* hdr, const uint32_t* ids, uint32_t* bucket_start,
                                  uint32_t V, uint32_t n_rows, uint32_t n_in_rows);
// Same, restricted to the message's input rows when input_rows_only != 0.
cudaError_t launch_apply_rows(const Launcher& L, const MsgHeader* hdr, const uint32_t* ids, const float* delta,
                              float* table, const Shape& s, int input_rows_only);

}  // namespace tensair
