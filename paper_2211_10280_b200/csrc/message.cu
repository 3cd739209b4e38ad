// Building the sparse gradient message from the row-sorted contributions, fused with the local
// gradient application of its output rows.
//
// After the stable sort all contributions to one row are contiguous and in a fixed order.  "Heads"
// (first item of each distinct key) give the message's ascending id list and the segment bounds.
// The scalars of the contributions are gathered into that order once ("terms").
// A warp then owns a row: it adds coefficient * source row over the segment (source = the centre's
// input row and coefficient g for an output row; source = a position's partial centre gradient and
// coefficient 1 for an input row), scales by -lr, writes the delta row into the message and, for an
// output row, adds it to the table in the same pass (as a bulk asynchronous add performed at the memory side).  Input rows are NOT updated here: they are the
// sources of every output-row sum and must keep their snapshot values until all sums are done.
// Rows with more than kChunk contributions are split into chunks that run on separate warps; their
// partial sums are combined in chunk order, so every sum has a fixed association.  All sums are
// accumulated in fp64 from the fp32 scalars and rows.
#include "kernels.h"

namespace tensair {

constexpr int kHeadThreads = 256;
constexpr int kHeadItems = 8;
constexpr int kHeadTile = kHeadThreads * kHeadItems;

uint32_t heads_tiles(uint32_t n_items) { return (n_items + kHeadTile - 1) / kHeadTile; }

__device__ inline uint32_t head_flags(const item_t* __restrict__ sorted, uint32_t n_items, uint32_t first,
                                      uint32_t keys[kHeadItems]) {
    uint32_t flags = 0;
    uint32_t prev = first > 0 && first <= n_items ? item_key(sorted[first - 1]) : 0xFFFFFFFFu;
#pragma unroll
    for (int i = 0; i < kHeadItems; ++i) {
        const uint32_t idx = first + i;
        keys[i] = idx < n_items ? item_key(sorted[idx]) : 0xFFFFFFFFu;
        if (idx < n_items && (idx == 0 || keys[i] != prev)) flags |= 1u << i;
        prev = keys[i];
    }
    return flags;
}

// Exclusive scan of the tile counts (in place), message header, reset of the long-row counters: the work of one
// block of kHeadThreads threads.
__device__ inline void scan_tile_counts(const item_t* __restrict__ sorted, uint32_t n_items, uint32_t V,
                                        uint32_t* tile_counts, uint32_t tiles, MsgHeader* __restrict__ hdr,
                                        uint32_t* __restrict__ seg_start, uint32_t* __restrict__ long_counters) {
    __shared__ uint32_t warp_tot[kHeadThreads / 32];
    __shared__ uint32_t carry_s;
    if (threadIdx.x == 0) {
        long_counters[0] = 0;
        long_counters[1] = 0;
        carry_s = 0;
    }
    __syncthreads();
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (uint32_t base = 0; base < tiles; base += kHeadThreads) {
        const uint32_t idx = base + threadIdx.x;
        const uint32_t v = idx < tiles ? __ldcg(tile_counts + idx) : 0;   // written by other blocks of this launch
        uint32_t incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= (uint32_t)o) incl += t;
        }
        if (lane == 31) warp_tot[wid] = incl;
        __syncthreads();
        uint32_t before = 0;
        for (uint32_t x = 0; x < wid; ++x) before += warp_tot[x];
        const uint32_t carry = carry_s;
        if (idx < tiles) tile_counts[idx] = carry + before + incl - v;
        __syncthreads();
        if (threadIdx.x == kHeadThreads - 1) carry_s = carry + before + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const uint32_t heads = carry_s;
        const bool dropped = n_items > 0 && item_key(sorted[n_items - 1]) == 2 * V;
        const uint32_t n_rows = heads - (dropped ? 1u : 0u);
        hdr->n_rows = n_rows;
        hdr->pad = 0;
        seg_start[heads] = n_items;
        if (!dropped) hdr->n_items = n_items;   // otherwise written by the head of the dropped run
    }
}

// Heads per tile; the block that finishes last (a ticket counts the blocks) scans the tile counts, so that no
// separate one-block launch stands between this kernel and the one that writes the heads.  Also the first kernel
// that runs once a batch is known to be valid as a whole: it adds the batch's tokens to the running unigram counts.
__global__ void __launch_bounds__(kHeadThreads)
k_heads_count(const item_t* __restrict__ sorted, uint32_t n_items, uint32_t V, uint32_t* tile_counts, uint32_t tiles,
              MsgHeader* __restrict__ hdr, uint32_t* __restrict__ seg_start, uint32_t* __restrict__ long_counters,
              const uint32_t* __restrict__ err, const int32_t* __restrict__ tok, uint32_t n,
              unsigned long long* __restrict__ counts, const uint8_t* __restrict__ owner) {
    if (*err) {
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            *hdr = MsgHeader{0, 0, 0, 0};
            long_counters[0] = 0;
            long_counters[1] = 0;
        }
        return;
    }
    __shared__ uint32_t warp_sum[kHeadThreads / 32];
    __shared__ uint32_t last_s;
    if (counts) {
        const uint32_t q = blockIdx.x * kHeadThreads + threadIdx.x;      // there are at least as many items as tokens
        if (q < n && (!owner || owner[q])) atomicAdd(counts + (uint32_t)tok[q], 1ULL);
    }
    uint32_t keys[kHeadItems];
    const uint32_t first = blockIdx.x * kHeadTile + threadIdx.x * kHeadItems;
    uint32_t c = __popc(head_flags(sorted, n_items, first, keys));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xFFFFFFFFu, c, o);
    if ((threadIdx.x & 31) == 0) warp_sum[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
        for (int i = 0; i < kHeadThreads / 32; ++i) t += warp_sum[i];
        tile_counts[blockIdx.x] = t;
        __threadfence();                                       // the count is visible before the ticket is taken
        last_s = atomicAdd(long_counters + 2, 1u) == tiles - 1 ? 1u : 0u;
    }
    __syncthreads();
    if (!last_s) return;
    __threadfence();
    if (threadIdx.x == 0) long_counters[2] = 0;                // ready for the next batch
    scan_tile_counts(sorted, n_items, V, tile_counts, tiles, hdr, seg_start, long_counters);
}

__global__ void __launch_bounds__(kHeadThreads)
k_heads_write(const item_t* __restrict__ sorted, uint32_t n_items, uint32_t V, const uint32_t* __restrict__ tile_base,
              MsgHeader* __restrict__ hdr, uint32_t* __restrict__ ids, uint32_t* __restrict__ seg_start,
              const Rec* __restrict__ rec, Rec* __restrict__ terms, const uint32_t* __restrict__ err,
              uint32_t* __restrict__ long_counters, LongRow* __restrict__ long_rows, ChunkItem* __restrict__ chunk_items,
              Limits lim) {
    if (*err) return;
    // terms[i] = scalar and centre token of the i-th sorted contribution (for an input-row item: the
    // centre position), so that the row sums read their terms contiguously
    for (uint32_t i = blockIdx.x * kHeadTile + threadIdx.x; i < n_items && i < (blockIdx.x + 1) * kHeadTile; i += kHeadThreads) {
        const item_t it = sorted[i];
        const uint32_t key = item_key(it);
        if (key < V) terms[i] = Rec{1.0, item_payload(it), 0u};
        else if (key < 2 * V && in_bounds(lim, item_payload(it), lim.contrib)) terms[i] = rec[item_payload(it)];
    }
    __shared__ uint32_t warp_tot[kHeadThreads / 32];
    uint32_t keys[kHeadItems];
    const uint32_t first = blockIdx.x * kHeadTile + threadIdx.x * kHeadItems;
    const uint32_t flags = head_flags(sorted, n_items, first, keys);
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t c = __popc(flags);
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= (uint32_t)o) incl += t;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    uint32_t m = tile_base[blockIdx.x] + incl - c;
    for (uint32_t x = 0; x < wid; ++x) m += warp_tot[x];
    uint32_t prev = first > 0 && first <= n_items ? item_key(sorted[first - 1]) : 0u;
#pragma unroll
    for (int i = 0; i < kHeadItems; ++i) {
        if ((flags & (1u << i)) && in_bounds(lim, m, (uint64_t)lim.batch_rows + 1)) {
            const uint32_t key = keys[i];
            const uint32_t start = first + i;
            seg_start[m] = start;
            if (key < 2 * V) ids[m] = key;
            else hdr->n_items = start;                           // first dropped negative
            if (key >= V && (start == 0 || prev < V)) hdr->n_in_rows = m;   // first output row
            // A row with more than kChunk contributions goes on the long-row list, cut into chunks (the order of the
            // lists does not reach any sum).  Its end is the upper bound of its key among the sorted items; only the
            // few long rows pay for that search.
            const uint32_t probe = start + kChunk;
            if (key < 2 * V && probe < n_items && item_key(sorted[probe]) == key) {
                uint32_t lo = probe + 1, hi = n_items;
                while (lo < hi) {
                    const uint32_t mid = lo + ((hi - lo) >> 1);
                    if (item_key(sorted[mid]) <= key) lo = mid + 1; else hi = mid;
                }
                const uint32_t nch = (lo - start + kChunk - 1) / kChunk;
                const uint32_t slot = atomicAdd(long_counters, 1u);
                const uint32_t base = atomicAdd(long_counters + 1, nch);
                if (in_bounds(lim, slot, lim.long_rows) && in_bounds(lim, (uint64_t)base + nch - 1, lim.chunks)) {
                    long_rows[slot] = LongRow{m, base, nch};
                    for (uint32_t ch = 0; ch < nch; ++ch) chunk_items[base + ch] = ChunkItem{m, ch};
                }
            }
            ++m;
        }
        prev = keys[i];
    }
}

cudaError_t launch_heads(const Launcher& L, const item_t* sorted, uint32_t n_items, uint32_t V, uint32_t* tile_counts,
                         MsgHeader* hdr, uint32_t* ids, uint32_t* seg_start, uint32_t* long_counters,
                         const Rec* rec, Rec* terms, const uint32_t* err, LongRow* long_rows, ChunkItem* chunk_items,
                         const int32_t* tok, uint32_t n, unsigned long long* counts, const uint8_t* owner) {
    const uint32_t tiles = heads_tiles(n_items);
    if (!tiles) return cudaSuccess;
    {
        Timed timed(L, K_HEADS_COUNT);
        k_heads_count<<<tiles, kHeadThreads, 0, L.stream>>>(sorted, n_items, V, tile_counts, tiles, hdr, seg_start,
                                                            long_counters, err, tok, n, counts, owner);
    }
    if (tiles) {
        Timed timed(L, K_HEADS_WRITE);
        k_heads_write<<<tiles, kHeadThreads, 0, L.stream>>>(sorted, n_items, V, tile_counts, hdr, ids, seg_start, rec, terms, err,
                                                            long_counters, long_rows, chunk_items, L.lim);
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// per-row sums
// ---------------------------------------------------------------------------------------------
constexpr int kTermsInFlightRows = 1;     // source rows a warp of the row kernel gathers at once (few: more warps fit)
constexpr int kTermsInFlightChunks = 4;   // the same for the chunk kernel, whose segments are long
constexpr int kReduceThreads = 128;

// One lane's share of a row sum: fp64 accumulators for its NV float4 slices.
template <int NV>
struct RowSum {
    double a[NV][4];
    __device__ inline void clear() {
#pragma unroll
        for (int i = 0; i < NV; ++i) a[i][0] = a[i][1] = a[i][2] = a[i][3] = 0.0;
    }
};

// Adds coefficient * source over terms[beg, end) in order.  A warp fetches up to 32 terms with one
// coalesced load and hands them round by shuffle; the fp32 source rows of four terms are in flight
// together.  Products and sums are taken in fp64, so the result does not feel the cancellation
// between the positive and negative terms of a row.
template <int NV, int kTermsInFlight>
__device__ inline void accumulate_segment(const Rec* __restrict__ terms, uint32_t beg, uint32_t end, bool input_row,
                                          const double* __restrict__ gin_pos, const float4* __restrict__ table,
                                          uint32_t d4, uint32_t stride4, uint32_t lane, RowSum<NV>& sum, const Limits& lim,
                                          bool have_first = false, Rec first = Rec{0.0, 0u, 0u}) {
    for (uint32_t base = beg; base < end; base += 32) {
        const uint32_t cnt = end - base < 32 ? end - base : 32;
        Rec mine = Rec{0.0, 0u, 0u};
        if (have_first && base == beg) mine = first;   // the caller fetched the first 32 terms ahead of time
        else if (lane < cnt) mine = terms[base + lane];
        if (input_row) {
            // Sources are the fp64 partial centre gradients of the positions holding this token.
            if constexpr (kTermsInFlight == 1) {
                for (uint32_t t = 0; t < cnt; ++t) {
                    const uint32_t q = __shfl_sync(0xFFFFFFFFu, mine.centre, t);
                    if (!in_bounds(lim, q, lim.positions)) continue;
                    const double2* src = reinterpret_cast<const double2*>(gin_pos + (size_t)q * stride4 * 4);
#pragma unroll
                    for (int j = 0; j < NV; ++j) {
                        const uint32_t e = lane + 32 * j;
                        if (e < d4) {
                            const double2 lo = src[2 * e], hi = src[2 * e + 1];
                            sum.a[j][0] += lo.x; sum.a[j][1] += lo.y; sum.a[j][2] += hi.x; sum.a[j][3] += hi.y;
                        }
                    }
                }
            } else {
                // The chunk kernel, whose segments are long, fetches the rows of several terms before any is added
                // (in term order), so that several loads are in flight, not one; how many, the row width decides.
                constexpr int kAhead = NV <= 2 ? 4 : (NV <= 4 ? 2 : 1);
                for (uint32_t t0 = 0; t0 < cnt; t0 += kAhead) {
                    double2 part[kAhead][NV][2];
#pragma unroll
                    for (int t = 0; t < kAhead; ++t) {
                        const uint32_t q = __shfl_sync(0xFFFFFFFFu, mine.centre, (t0 + t) & 31);
                        const double2* src = reinterpret_cast<const double2*>(gin_pos + (size_t)q * stride4 * 4);
#pragma unroll
                        for (int j = 0; j < NV; ++j) {
                            const uint32_t e = lane + 32 * j;
                            const bool on = t0 + t < cnt && e < d4 && in_bounds(lim, q, lim.positions);
                            part[t][j][0] = on ? src[2 * e] : make_double2(0.0, 0.0);
                            part[t][j][1] = on ? src[2 * e + 1] : make_double2(0.0, 0.0);
                        }
                    }
#pragma unroll
                    for (int t = 0; t < kAhead; ++t) {
                        if (t0 + t < cnt) {
#pragma unroll
                            for (int j = 0; j < NV; ++j) {
                                sum.a[j][0] += part[t][j][0].x; sum.a[j][1] += part[t][j][0].y;
                                sum.a[j][2] += part[t][j][1].x; sum.a[j][3] += part[t][j][1].y;
                            }
                        }
                    }
                }
            }
            continue;
        }
        for (uint32_t t0 = 0; t0 < cnt; t0 += kTermsInFlight) {
            const float4* src[kTermsInFlight];
            double coef[kTermsInFlight];
#pragma unroll
            for (int t = 0; t < kTermsInFlight; ++t) {
                const uint32_t from = (t0 + t) & 31;
                const double g = __shfl_sync(0xFFFFFFFFu, mine.g, from);
                const uint32_t centre = __shfl_sync(0xFFFFFFFFu, mine.centre, from);
                const bool on = t0 + t < cnt && in_bounds(lim, centre, lim.table_rows / 2);
                coef[t] = on ? g * kWidenUp : 0.0;   // exact (|g| <= 1); the factor the widened source lacks
                src[t] = table + (size_t)(on ? centre : 0u) * stride4;
            }
            float4 x[kTermsInFlight][NV];
#pragma unroll
            for (int t = 0; t < kTermsInFlight; ++t)
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const uint32_t e = lane + 32 * i;
                    x[t][i] = (t0 + t < cnt && e < d4) ? src[t][e] : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
            for (int t = 0; t < kTermsInFlight; ++t)
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    sum.a[i][0] = fma(coef[t], widen_down(x[t][i].x), sum.a[i][0]);
                    sum.a[i][1] = fma(coef[t], widen_down(x[t][i].y), sum.a[i][1]);
                    sum.a[i][2] = fma(coef[t], widen_down(x[t][i].z), sum.a[i][2]);
                    sum.a[i][3] = fma(coef[t], widen_down(x[t][i].w), sum.a[i][3]);
                }
        }
    }
}

// The table row of an output id, fetched before the sum starts so that its latency hides behind the sum.
template <int NV>
struct RowPrefetch {
    float4 r[NV];
    __device__ inline void load(const float4* __restrict__ table, uint32_t id, uint32_t V, uint32_t d4, uint32_t stride4,
                                uint32_t lane) {
        if (id >= V) {
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const uint32_t e = lane + 32 * i;
                if (e < d4) r[i] = table[(size_t)id * stride4 + e];
            }
        }
    }
};

// delta = fp32(-scale * sum); the delta row goes into the message and, for an output row, onto the table.
template <int NV>
__device__ inline void finish_row(const RowSum<NV>& sum, const RowPrefetch<NV>& old, uint32_t m, uint32_t id, uint32_t V,
                                  double scale, float4* __restrict__ table, float4* __restrict__ delta, uint32_t d4,
                                  uint32_t stride4, uint32_t lane) {
    const double nlr = -scale;
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const uint32_t e = lane + 32 * i;
        if (e < d4) {
            const float4 dl = make_float4((float)(nlr * sum.a[i][0]), (float)(nlr * sum.a[i][1]),
                                          (float)(nlr * sum.a[i][2]), (float)(nlr * sum.a[i][3]));
            delta[(size_t)m * stride4 + e] = dl;
            if (id >= V) {
                float4 t = old.r[i];
                t.x += dl.x; t.y += dl.y; t.z += dl.z; t.w += dl.w;
                table[(size_t)id * stride4 + e] = t;
            }
        }
    }
}

// ---- bulk asynchronous copies out of shared memory -------------------------------------------------
__device__ inline uint32_t smem_addr32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// Makes this thread's earlier shared-memory writes visible to the asynchronous copy engine.
__device__ inline void fence_smem_writes_for_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// global[dst .. dst+bytes) = shared[src .. src+bytes)
__device__ inline void bulk_store_s2g(void* dst_global, const void* src_smem, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(dst_global), "r"(smem_addr32(src_smem)), "r"(bytes) : "memory");
}
// global[dst + i] += shared[src + i] for every fp32 element: the read-modify-write is done at the memory
// side (one IEEE addition per element, rounded to nearest even; each destination row has one writer here).
__device__ inline void bulk_add_f32_s2g(void* dst_global, const void* src_smem, uint32_t bytes) {
    asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;"
                 ::"l"(dst_global), "r"(smem_addr32(src_smem)), "r"(bytes) : "memory");
}
__device__ inline void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until all but the newest `keep` groups of this thread have finished READING their shared-memory source.
template <int keep>
__device__ inline void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(keep) : "memory"); }
__device__ inline void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

constexpr int kOutBuffers = 2;   // delta rows a warp may have on their way out

// One warp per message row, rows taken in a grid-stride loop that is software-pipelined: while row i is
// summed, the terms of row i+1 and the segment bounds of row i+2 are already on their way.  The finished
// delta row is placed in shared memory and leaves by two bulk asynchronous operations: a store into the
// message and, for an output row, an add onto the table row.  The table row is never read into the
// multiprocessor, so nothing here waits on DRAM.
template <int NV>
__global__ void __launch_bounds__(kReduceThreads)
k_reduce_rows(const Rec* __restrict__ terms, const MsgHeader* __restrict__ hdr, const uint32_t* __restrict__ ids,
              const uint32_t* __restrict__ seg_start, const double* __restrict__ gin_pos,
              float4* __restrict__ table, float4* __restrict__ delta, uint32_t V, uint32_t d4, uint32_t stride4,
              double scale, Limits lim) {
    extern __shared__ __align__(128) float4 out_rows[];   // [warps in block][kOutBuffers][stride4]
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    float4* my_out = out_rows + (size_t)(threadIdx.x >> 5) * kOutBuffers * stride4;
    const uint32_t n_rows = hdr->n_rows;
    if (!in_bounds(lim, n_rows, (uint64_t)lim.batch_rows + 1)) return;
    const uint32_t row_bytes = d4 * 16;
    const double nscale = -scale;
    struct Meta { uint32_t beg, end, id; };
    auto load_meta = [&](uint32_t m) {
        Meta x{0u, 0u, 0u};
        if (m < n_rows) { x.beg = seg_start[m]; x.end = seg_start[m + 1]; x.id = ids[m]; }
        return x;
    };
    auto load_terms = [&](const Meta& x) {
        Rec r{0.0, 0u, 0u};
        if (x.end - x.beg <= kChunk && x.beg + lane < x.end) r = terms[x.beg + lane];
        return r;
    };
    uint32_t m = warp;
    Meta cur = load_meta(m), nxt = load_meta(m + nwarps);
    Rec cur_terms = load_terms(cur);
    uint32_t buf = 0;
    for (; m < n_rows; m += nwarps) {
        const Meta after = load_meta(m + 2 * nwarps);
        const Rec nxt_terms = load_terms(nxt);
        if (cur.end - cur.beg <= kChunk) {   // longer rows are on the long-row list and summed by the chunk kernels
            RowSum<NV> sum;
            sum.clear();
            accumulate_segment<NV, kTermsInFlightRows>(terms, cur.beg, cur.end, cur.id < V, gin_pos, table, d4, stride4, lane, sum, lim,
                                   true, cur_terms);
            // the buffer about to be refilled must have been read by the copies issued from it
            if (lane == 0) bulk_wait_read<kOutBuffers - 1>();
            __syncwarp();
            float4* out = my_out + (size_t)buf * stride4;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const uint32_t e = lane + 32 * i;
                if (e < d4)
                    out[e] = make_float4((float)(nscale * sum.a[i][0]), (float)(nscale * sum.a[i][1]),
                                         (float)(nscale * sum.a[i][2]), (float)(nscale * sum.a[i][3]));
            }
            fence_smem_writes_for_async();
            __syncwarp();
            if (lane == 0 && in_bounds(lim, m, lim.slot_rows) && in_bounds(lim, cur.id, lim.table_rows)) {
                bulk_store_s2g(delta + (size_t)m * stride4, out, row_bytes);
                if (cur.id >= V) bulk_add_f32_s2g(table + (size_t)cur.id * stride4, out, row_bytes);
                bulk_commit();
            }
            buf = (buf + 1) % kOutBuffers;
        }
        cur = nxt;
        nxt = after;
        cur_terms = nxt_terms;
    }
    if (lane == 0) bulk_wait_all();
}

// Partial sums of the chunks of long rows, one warp per chunk; partials are kept in fp64.
template <int NV>
__global__ void __launch_bounds__(kReduceThreads)
k_reduce_chunks(const Rec* __restrict__ terms, const uint32_t* __restrict__ ids, const uint32_t* __restrict__ seg_start,
                const double* __restrict__ gin_pos, const float4* __restrict__ table,
                uint32_t V, uint32_t d4, uint32_t stride4, const uint32_t* __restrict__ long_counters,
                const ChunkItem* __restrict__ chunk_items, double* __restrict__ partials, Limits lim) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t n_chunks = long_counters[1];
    if (!in_bounds(lim, n_chunks, (uint64_t)lim.chunks + 1)) return;
    for (uint32_t x = warp; x < n_chunks; x += nwarps) {
        const ChunkItem ci = chunk_items[x];
        if (!in_bounds(lim, ci.m, lim.batch_rows)) continue;
        const uint32_t beg = seg_start[ci.m] + ci.chunk * kChunk;
        const uint32_t seg_end = seg_start[ci.m + 1];
        const uint32_t end = beg + kChunk < seg_end ? beg + kChunk : seg_end;
        RowSum<NV> sum;
        sum.clear();
        accumulate_segment<NV, kTermsInFlightChunks>(terms, beg, end, ids[ci.m] < V, gin_pos, table, d4, stride4, lane, sum, lim);
        double* out = partials + (size_t)x * stride4 * 4;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const uint32_t e = lane + 32 * i;
            if (e < d4) {
                reinterpret_cast<double2*>(out)[2 * e] = make_double2(sum.a[i][0], sum.a[i][1]);
                reinterpret_cast<double2*>(out)[2 * e + 1] = make_double2(sum.a[i][2], sum.a[i][3]);
            }
        }
    }
}

// Long rows: one block per row.  Warp w adds a contiguous run of the row's chunk partials in chunk order
// (four fetched together), the runs are then added in warp order by warp 0, and the row is finished like a
// short one - a fixed association for every launch shape.
constexpr int kLongWarps = 8;
template <int NV>
__global__ void __launch_bounds__(kLongWarps * 32)
k_reduce_long(const uint32_t* __restrict__ ids, const double* __restrict__ partials, float4* __restrict__ table,
              float4* __restrict__ delta, uint32_t V, uint32_t d4, uint32_t stride4, double scale,
              const uint32_t* __restrict__ long_counters, const LongRow* __restrict__ long_rows, uint32_t warps, Limits lim) {
    extern __shared__ __align__(16) double runs[];   // [warps][4 * d4]
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const uint32_t n_long = long_counters[0];
    if (!in_bounds(lim, n_long, (uint64_t)lim.long_rows + 1)) return;
    for (uint32_t x = blockIdx.x; x < n_long; x += gridDim.x) {
        const LongRow row = long_rows[x];
        // block-uniform: every thread sees the same row record
        if (!in_bounds(lim, row.m, lim.batch_rows) || !in_bounds(lim, (uint64_t)row.base + row.nchunks, (uint64_t)lim.chunks + 1)) continue;
        const uint32_t id = ids[row.m];
        if (!in_bounds(lim, id, lim.table_rows) || !in_bounds(lim, row.m, lim.slot_rows)) continue;
        const uint32_t per = (row.nchunks + warps - 1) / warps;
        const uint32_t c_beg = wid * per < row.nchunks ? wid * per : row.nchunks;
        const uint32_t c_end = c_beg + per < row.nchunks ? c_beg + per : row.nchunks;
        RowSum<NV> sum;
        sum.clear();
        for (uint32_t c0 = c_beg; c0 < c_end; c0 += 4) {
            double2 part[4][NV][2];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const double2* in = reinterpret_cast<const double2*>(partials + (size_t)(row.base + c0 + t) * stride4 * 4);
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const uint32_t e = lane + 32 * i;
                    const bool on = c0 + t < c_end && e < d4;
                    part[t][i][0] = on ? in[2 * e] : make_double2(0.0, 0.0);
                    part[t][i][1] = on ? in[2 * e + 1] : make_double2(0.0, 0.0);
                }
            }
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    sum.a[i][0] += part[t][i][0].x; sum.a[i][1] += part[t][i][0].y;
                    sum.a[i][2] += part[t][i][1].x; sum.a[i][3] += part[t][i][1].y;
                }
        }
        double2* mine = reinterpret_cast<double2*>(runs + (size_t)wid * d4 * 4);
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const uint32_t e = lane + 32 * i;
            if (e < d4) {
                mine[2 * e] = make_double2(sum.a[i][0], sum.a[i][1]);
                mine[2 * e + 1] = make_double2(sum.a[i][2], sum.a[i][3]);
            }
        }
        __syncthreads();
        if (wid == 0) {
            RowPrefetch<NV> old;
            old.load(table, id, V, d4, stride4, lane);
            for (uint32_t w = 1; w < warps; ++w) {
                const double2* other = reinterpret_cast<const double2*>(runs + (size_t)w * d4 * 4);
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const uint32_t e = lane + 32 * i;
                    if (e < d4) {
                        const double2 lo = other[2 * e], hi = other[2 * e + 1];
                        sum.a[i][0] += lo.x; sum.a[i][1] += lo.y; sum.a[i][2] += hi.x; sum.a[i][3] += hi.y;
                    }
                }
            }
            finish_row<NV>(sum, old, row.m, id, V, scale, table, delta, d4, stride4, lane);
        }
        __syncthreads();
    }
}

template <int NV>
static cudaError_t reduce_short(const Launcher& L, const Rec* terms, const MsgHeader* hdr, const uint32_t* ids,
                                const uint32_t* seg_start, const double* gin_pos, float* table, float* delta,
                                const Shape& s, double scale) {
    const uint32_t stride4 = s.stride / 4;
    const size_t out_smem = (size_t)(kReduceThreads / 32) * kOutBuffers * s.stride * 4;
    Timed timed(L, K_REDUCE_ROWS);
    k_reduce_rows<NV><<<L.sms * grid_shape().reduce_blocks_per_sm, kReduceThreads, out_smem, L.stream>>>(
        terms, hdr, ids, seg_start, gin_pos, reinterpret_cast<float4*>(table), reinterpret_cast<float4*>(delta), s.V, s.d4,
        stride4, scale, L.lim);
    return cudaGetLastError();
}

template <int NV>
static cudaError_t reduce_listed(const Launcher& L, const Rec* terms, const uint32_t* ids, const uint32_t* seg_start,
                                 const double* gin_pos, float* table, float* delta, const Shape& s, double scale,
                                 const uint32_t* long_counters, const LongRow* long_rows, const ChunkItem* chunk_items,
                                 double* partials) {
    const uint32_t stride4 = s.stride / 4;
    float4* t4 = reinterpret_cast<float4*>(table);
    float4* d4p = reinterpret_cast<float4*>(delta);
    {
        Timed timed(L, K_REDUCE_CHUNKS);
        k_reduce_chunks<NV><<<L.sms * grid_shape().reduce_blocks_per_sm, kReduceThreads, 0, L.stream>>>(
            terms, ids, seg_start, gin_pos, t4, s.V, s.d4, stride4, long_counters, chunk_items, partials, L.lim);
    }
    {
        Timed timed(L, K_REDUCE_LONG);
        uint32_t long_warps = 49152 / (s.d * 8);          // run sums of one block within 48 KB of shared memory
        if (long_warps > (uint32_t)kLongWarps) long_warps = kLongWarps;
        if (long_warps < 1) long_warps = 1;
        k_reduce_long<NV><<<L.sms * 2, long_warps * 32, (size_t)long_warps * s.d * 8, L.stream>>>(
            ids, partials, t4, d4p, s.V, s.d4, stride4, scale, long_counters, long_rows, long_warps, L.lim);
    }
    return cudaGetLastError();
}

#define TENSAIR_BY_WIDTH(CALL)            \
    if (s.d4 <= 32) return CALL(1);       \
    if (s.d4 <= 64) return CALL(2);       \
    if (s.d4 <= 96) return CALL(3);       \
    if (s.d4 <= 128) return CALL(4);      \
    return CALL(8)

// Rows with at most kChunk contributions: summed, written into the message and (output rows) added to the table.
cudaError_t launch_reduce_rows(const Launcher& L, const Rec* terms, const MsgHeader* hdr, const uint32_t* ids,
                               const uint32_t* seg_start, const double* gin_pos, float* table, float* delta,
                               const Shape& s, double scale) {
#define TENSAIR_CALL(NV) reduce_short<NV>(L, terms, hdr, ids, seg_start, gin_pos, table, delta, s, scale)
    TENSAIR_BY_WIDTH(TENSAIR_CALL);
#undef TENSAIR_CALL
}

// The listed long rows: chunk partials, then one block per row.  Touches none of the rows the kernel above
// writes and reads nothing it writes, so the two may run side by side.
cudaError_t launch_reduce_long_rows(const Launcher& L, const Rec* terms, const uint32_t* ids, const uint32_t* seg_start,
                                    const double* gin_pos, float* table, float* delta, const Shape& s, double scale,
                                    const uint32_t* long_counters, const LongRow* long_rows,
                                    const ChunkItem* chunk_items, double* partials) {
#define TENSAIR_CALL(NV) \
    reduce_listed<NV>(L, terms, ids, seg_start, gin_pos, table, delta, s, scale, long_counters, long_rows, chunk_items, partials)
    TENSAIR_BY_WIDTH(TENSAIR_CALL);
#undef TENSAIR_CALL
}
#undef TENSAIR_BY_WIDTH

}  // namespace tensair
