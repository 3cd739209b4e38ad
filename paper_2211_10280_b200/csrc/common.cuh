// Shared device-side definitions of the SGNS / DASGD kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace tensair {

// One sort item: key (row id in the unified [0,2V) space, or 2V for a dropped negative) in the
// high word, payload in the low word.  Payload: the centre position q for an input-row item, the
// contribution index c = p*(k+1)+j for an output-row item.
typedef unsigned long long item_t;
__host__ __device__ inline uint32_t item_key(item_t it) { return (uint32_t)(it >> 32); }
__host__ __device__ inline uint32_t item_payload(item_t it) { return (uint32_t)it; }
__host__ __device__ inline item_t make_item(uint32_t key, uint32_t payload) {
    return ((item_t)key << 32) | payload;
}

// Gradient scalar of one contribution and the centre token whose input row it multiplies.
struct Rec {
    double g;
    uint32_t centre;
    uint32_t pad;
};

// Message slot header (the slot is: header, ids, delta rows).
struct MsgHeader {
    uint32_t n_rows;     // distinct touched rows
    uint32_t n_in_rows;  // of which input rows
    uint32_t n_items;    // sort items that are not dropped negatives
    uint32_t pad;
};
constexpr uint32_t kHeaderBytes = 256;
// Every message carries an index of its rows by id range ("bucket" b = ids in [b << kBucketShift, (b+1) << kBucketShift)):
// bucket_start[b] = first row whose id is not below the bucket.  It lets one pass apply several messages
// id range by id range, so that a table row touched by more than one of them is fetched from memory once.
constexpr uint32_t kBucketShift = 4;
__host__ __device__ inline uint32_t bucket_count(uint32_t V) { return ((2 * V - 1) >> kBucketShift) + 1; }

// A long row (more contributions than one warp takes in one go) and its chunk partials.
struct LongRow {
    uint32_t m;          // message row index
    uint32_t base;       // first partial slot
    uint32_t nchunks;
};
struct ChunkItem {
    uint32_t m;
    uint32_t chunk;
};
constexpr uint32_t kChunk = 64;    // contributions per chunk; rows with more than this go the long way

// Sum over i < x of min(i, w): how many left (or, mirrored, right) neighbours the first x positions have.
__host__ __device__ inline uint64_t neighbours_before(uint64_t x, uint64_t w) {
    return x <= w + 1 ? x * (x - (x ? 1 : 0)) / 2 : w * (w + 1) / 2 + (x - w - 1) * w;
}
// Index of the first pair of centre position q in a batch of n tokens with window w,
// pairs enumerated by (q ascending, context position ascending).
__host__ __device__ inline uint32_t pair_offset(uint32_t q, uint32_t n, uint32_t w) {
    return (uint32_t)(neighbours_before(q, w) + neighbours_before(n, w) - neighbours_before(n - q, w));
}
__host__ __device__ inline uint32_t pair_count(uint32_t n, uint32_t w) {
    return (uint32_t)(2 * neighbours_before(n, w));
}

// fp32 -> fp64 without the conversion unit.  A finite float with sign s, exponent field e and fraction m, read
// as the double with the same sign, exponent field e (not re-biased) and fraction m << 29, is f * 2^-896 exactly:
// normal, subnormal and zero alike.  The bits come from one sign-extending shift of the float's word by 29 places
// and one mask; the factor 2^896 goes, exactly, into the other operand of the product the value enters.
// Infinities and NaNs are not preserved (they read as finite values): table rows must be finite.
__device__ inline double widen_down(float f) {
    const long long w = (long long)__float_as_int(f) << 29;
    return __hiloint2double((int)(w >> 32) & (int)0x8FFFFFFFu, (int)w);
}
constexpr double kWidenUp = 0x1p896;   // widen_down(f) * kWidenUp == (double)f

// Bits of the device error word (sticky until a synchronising call reads and clears it).
constexpr uint32_t kErrBadToken = 1u;   // a batch held a token id outside [0,V)
constexpr uint32_t kErrTimeout = 2u;    // a bounded wait for a warp's own bulk copies ran out
constexpr uint32_t kErrBounds = 4u;     // checked build: an index left its array; the access was skipped
constexpr uint32_t kErrOverflow = 8u;   // a merged message had more rows than its slot holds; the rest was dropped

// Sizes of the arrays that kernels index with values computed from data.  In a checked build (-DTENSAIR_BOUNDS)
// every such index is compared with its bound first; one out of bounds raises kErrBounds in the error word and the
// access is skipped - nothing traps.  In a normal build the checks compile to nothing.
struct Limits {
    uint32_t* err;
    uint32_t table_rows;   // 2V rows of one replica's unified table
    uint32_t slot_rows;    // rows a message slot holds
    uint32_t batch_rows;   // rows the message of one batch can have (bounds the per-batch segment list)
    uint32_t items;        // sort items of a batch
    uint32_t contrib;      // contributions of a batch (row ids, gradient scalars)
    uint32_t positions;    // partial centre gradients of a batch: two per position
    uint32_t long_rows;    // entries of the long-row list
    uint32_t chunks;       // entries of the chunk list and of the chunk partials
};
#ifdef TENSAIR_BOUNDS
__device__ inline bool in_bounds(const Limits& lim, uint64_t index, uint64_t bound) {
    if (index < bound) return true;
    atomicOr(lim.err, kErrBounds);
    return false;
}
#else
__device__ __forceinline__ bool in_bounds(const Limits&, uint64_t, uint64_t) { return true; }
#endif

struct Shape {
    uint32_t V, d, d4, stride, w, k, K1;
};

}  // namespace tensair
