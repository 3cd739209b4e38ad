// Gradient application of a sparse message: table[id] += delta for every row of the message.
//
// Pure streaming scatter-add: the delta rows are contiguous, the ids ascend, so the table rows are
// visited in address order.  One warp per row, 128-bit accesses, rows taken in a grid-stride loop
// by a grid sized to the machine; the row count is read from the message header on the device.
#include "kernels.h"

namespace tensair {

GridShape& grid_shape() {
    static GridShape shape;
    return shape;
}

template <int NV>
__global__ void __launch_bounds__(256)
k_apply(const MsgHeader* __restrict__ hdr, const uint32_t* __restrict__ ids, const float4* __restrict__ delta,
        float4* __restrict__ table, uint32_t d4, uint32_t stride4, int input_rows_only, Limits lim) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t limit = input_rows_only ? hdr->n_in_rows : hdr->n_rows;
    if (!in_bounds(lim, limit, (uint64_t)lim.slot_rows + 1)) return;
    for (uint32_t m = warp; m < limit; m += nwarps) {
        const uint32_t id = __ldg(ids + m);
        if (!in_bounds(lim, id, lim.table_rows)) continue;
        const float4* __restrict__ src = delta + (size_t)m * stride4;
        float4* __restrict__ dst = table + (size_t)id * stride4;
        float4 a[NV], b[NV];
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const uint32_t e = lane + 32 * i;
            if (e < d4) {
                a[i] = __ldg(src + e);
                b[i] = dst[e];
            }
        }
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const uint32_t e = lane + 32 * i;
            if (e < d4) {
                b[i].x += a[i].x; b[i].y += a[i].y; b[i].z += a[i].z; b[i].w += a[i].w;
                dst[e] = b[i];
            }
        }
    }
}

cudaError_t launch_apply_rows(const Launcher& L, const MsgHeader* hdr, const uint32_t* ids, const float* delta,
                              float* table, const Shape& s, int input_rows_only) {
    const uint32_t stride4 = s.stride / 4;
    const float4* d4p = reinterpret_cast<const float4*>(delta);
    float4* t4 = reinterpret_cast<float4*>(table);
    Timed timed(L, input_rows_only ? K_APPLY_INPUT_ROWS : K_APPLY_MESSAGE);
#define TENSAIR_APPLY(NV)                                                                 \
    k_apply<NV><<<L.sms * grid_shape().apply_blocks_per_sm, 256, 0, L.stream>>>(hdr, ids, d4p, t4, s.d4, stride4, \
                                                                               input_rows_only, L.lim)
    if (s.d4 <= 32) TENSAIR_APPLY(1);
    else if (s.d4 <= 64) TENSAIR_APPLY(2);
    else if (s.d4 <= 96) TENSAIR_APPLY(3);
    else if (s.d4 <= 128) TENSAIR_APPLY(4);
    else TENSAIR_APPLY(8);
#undef TENSAIR_APPLY
    return cudaGetLastError();
}

// One thread per bucket boundary: lower bound of b << kBucketShift in the ascending id list.  One block more than the
// boundaries need adds up the batch's loss (the per-half-position losses in a fixed order, in fp64; in a routed
// batch only the replica's own positions): both are small, independent of each other and wanted at the same point of
// the batch, so they share a launch.
__global__ void __launch_bounds__(256)
k_bucket_index(const MsgHeader* __restrict__ hdr, const uint32_t* __restrict__ ids, uint32_t* __restrict__ bucket_start,
               uint32_t n_buckets, const double* __restrict__ loss_pos, uint32_t n_loss, double* __restrict__ loss,
               const uint32_t* __restrict__ err, const uint8_t* __restrict__ owner) {
    if (loss && blockIdx.x == gridDim.x - 1) {
        // the association of the one-block loss kernel (1024 strided partial sums, then a binary tree), so that every
        // entry point reports the same bits
        __shared__ double part[1024];
        for (uint32_t t = threadIdx.x; t < 1024; t += 256) {
            double s = 0.0;
            if (!*err)
                for (uint32_t i = t; i < n_loss; i += 1024)
                    if (!owner || owner[i >> 1]) s += loss_pos[i];
            part[t] = s;
        }
        __syncthreads();
        for (uint32_t o = 512; o > 0; o >>= 1) {
            for (uint32_t t = threadIdx.x; t < o; t += 256) part[t] += part[t + o];
            __syncthreads();
        }
        if (threadIdx.x == 0) *loss = part[0];
        return;
    }
    const uint32_t b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b > n_buckets) return;
    const uint32_t n_rows = hdr->n_rows;
    const uint64_t key = (uint64_t)b << kBucketShift;
    uint32_t lo = 0, hi = n_rows;
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if ((uint64_t)__ldg(ids + mid) < key) lo = mid + 1; else hi = mid;
    }
    bucket_start[b] = lo;
}

cudaError_t launch_bucket_index(const Launcher& L, const MsgHeader* hdr, const uint32_t* ids, uint32_t* bucket_start,
                                uint32_t V, const double* loss_pos, uint32_t n, double* loss, const uint32_t* err,
                                const uint8_t* owner) {
    const uint32_t nb = bucket_count(V);
    Timed timed(L, K_BUCKET_INDEX);
    k_bucket_index<<<(nb + 1 + 255) / 256 + (loss ? 1 : 0), 256, 0, L.stream>>>(hdr, ids, bucket_start, nb, loss_pos,
                                                                               n < 2 ? 0 : 2 * n, loss, err, owner);
    return cudaGetLastError();
}

// The same index for a message whose rows arrived from another process: the row counts come from the host and
// are written into the slot's header here, so that the message reads like one built in place.
__global__ void __launch_bounds__(256)
k_index_received(MsgHeader* __restrict__ hdr, const uint32_t* __restrict__ ids, uint32_t* __restrict__ bucket_start,
                 uint32_t n_buckets, uint32_t n_rows, uint32_t n_in_rows) {
    const uint32_t b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0) *hdr = MsgHeader{n_rows, n_in_rows, 0u, 0u};
    if (b > n_buckets) return;
    const uint64_t key = (uint64_t)b << kBucketShift;
    uint32_t lo = 0, hi = n_rows;
    while (lo < hi) {
        const uint32_t mid = (lo + hi) >> 1;
        if ((uint64_t)__ldg(ids + mid) < key) lo = mid + 1; else hi = mid;
    }
    bucket_start[b] = lo;
}

cudaError_t launch_index_received(const Launcher& L, MsgHeader* hdr, const uint32_t* ids, uint32_t* bucket_start,
                                  uint32_t V, uint32_t n_rows, uint32_t n_in_rows) {
    const uint32_t nb = bucket_count(V);
    Timed timed(L, K_BUCKET_INDEX);
    k_index_received<<<(nb + 1 + 255) / 256, 256, 0, L.stream>>>(hdr, ids, bucket_start, nb, n_rows, n_in_rows);
    return cudaGetLastError();
}

// All receivers, one pass, no ordering barriers.  A message carries the set of receivers it is due for.  A block
// owns a bucket (16 consecutive row ids).  It first notes, per message, which of the 16 ids the message holds
// (a 16-bit mask; ids ascend, so the row of id j is the bucket's first row plus the number of mask bits below j).
// Then a warp takes one (id, receiver) pair at a time: it fetches the receiver's table row once, adds the delta
// rows of the messages that hold the id and are due for that receiver, in message order, and stores the row
// once.  The sums are the ones a message-after-message application makes (fp32 additions in the same order);
// a delta row needed by several receivers comes from memory once and from the cache afterwards.
static_assert(kBucketShift == 4, "the step kernel maps a bucket onto half a warp");
constexpr int kStepThreads = 128;
template <int NV>
__global__ void __launch_bounds__(kStepThreads)
k_apply_step(StepMessages f, uint32_t n_receivers, float4* __restrict__ tables, size_t replica4, uint32_t d4,
             uint32_t stride4, uint32_t n_buckets, Limits lim) {
    // two copies, used by alternate buckets: a warp may note the next bucket while another still works on this one
    __shared__ uint32_t first_row[2][kMaxStepMessages];
    __shared__ uint32_t held[2][kMaxStepMessages];
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    constexpr uint32_t kWarps = kStepThreads / 32;
    const uint32_t half = lane >> 4, j_mine = lane & 15;
    const uint32_t half_mask = 0xFFFFu << (16 * half);
    uint32_t turn = 0;
    for (uint32_t b = blockIdx.x; b < n_buckets; b += gridDim.x, turn ^= 1u) {
        // which ids of the bucket each message holds: half a warp per message
        for (uint32_t k0 = 2 * wid; k0 < f.count; k0 += 2 * kWarps) {
            const uint32_t k = k0 + half;
            uint32_t beg = 0, bit = 0;
            if (k < f.count) {
                beg = __ldg(f.buckets[k] + b);
                const uint32_t end = __ldg(f.buckets[k] + b + 1);
                if (beg + j_mine < end) bit = 1u << (__ldg(f.ids[k] + beg + j_mine) & 15u);
            }
            const uint32_t mask = __reduce_or_sync(half_mask, bit);
            if (k < f.count && j_mine == 0) { first_row[turn][k] = beg; held[turn][k] = mask; }
        }
        __syncthreads();
        const uint32_t set_mine = lane < f.count ? f.receivers[lane] : 0u;
        const uint32_t held_mine = lane < f.count ? held[turn][lane] : 0u;
        for (uint32_t task = wid; task < 16u * n_receivers; task += kWarps) {
            const uint32_t j = task / n_receivers, rcv = task - j * n_receivers;
            // messages (lane = message index, so in message order) that hold id j and are due for this receiver
            uint32_t todo = __ballot_sync(0xFFFFFFFFu, ((held_mine >> j) & 1u) && ((set_mine >> rcv) & 1u));
            if (!todo) continue;
            const uint32_t id = (b << kBucketShift) + j;
            if (!in_bounds(lim, id, lim.table_rows)) continue;
            float4* dst = tables + (size_t)rcv * replica4 + (size_t)id * stride4;
            float4 r[NV], a[NV];
            uint32_t k = (uint32_t)__ffs((int)todo) - 1u;
            todo &= todo - 1;
#ifdef TENSAIR_BOUNDS
            {   // every message that holds the id must hold it inside its slot
                bool inside = true;
                for (uint32_t rest = todo | (1u << k); rest; rest &= rest - 1) {
                    const uint32_t kk = (uint32_t)__ffs((int)rest) - 1u;
                    inside = inside && in_bounds(lim, first_row[turn][kk] + __popc(held[turn][kk] & ((1u << j) - 1u)), lim.slot_rows);
                }
                if (!inside) continue;
            }
#endif
            const float4* __restrict__ src = reinterpret_cast<const float4*>(f.delta[k]) +
                (size_t)(first_row[turn][k] + __popc(held[turn][k] & ((1u << j) - 1u))) * stride4;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const uint32_t e = lane + 32 * i;
                if (e < d4) {
                    r[i] = __ldcg(dst + e);
                    a[i] = __ldg(src + e);
                }
            }
            for (;;) {
#pragma unroll
                for (int i = 0; i < NV; ++i) { r[i].x += a[i].x; r[i].y += a[i].y; r[i].z += a[i].z; r[i].w += a[i].w; }
                if (!todo) break;
                k = (uint32_t)__ffs((int)todo) - 1u;
                todo &= todo - 1;
                src = reinterpret_cast<const float4*>(f.delta[k]) +
                      (size_t)(first_row[turn][k] + __popc(held[turn][k] & ((1u << j) - 1u))) * stride4;
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const uint32_t e = lane + 32 * i;
                    if (e < d4) a[i] = __ldg(src + e);
                }
            }
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const uint32_t e = lane + 32 * i;
                if (e < d4) dst[e] = r[i];
            }
        }
    }
}

cudaError_t launch_apply_step(const Launcher& L, const StepMessages& f, uint32_t n_receivers, float* tables,
                              size_t replica_floats, const Shape& s, int kind) {
    const uint32_t stride4 = s.stride / 4;
    float4* t4 = reinterpret_cast<float4*>(tables);
    const uint32_t nb = bucket_count(s.V);
    uint32_t blocks = (uint32_t)(L.sms * grid_shape().fused_blocks_per_sm);
    if (blocks > nb) blocks = nb;
    Timed timed(L, kind);
#define TENSAIR_STEP(NV) k_apply_step<NV><<<blocks, kStepThreads, 0, L.stream>>>(f, n_receivers, t4, replica_floats / 4, s.d4, stride4, nb, L.lim)
    if (s.d4 <= 32) TENSAIR_STEP(1);
    else if (s.d4 <= 64) TENSAIR_STEP(2);
    else if (s.d4 <= 96) TENSAIR_STEP(3);
    else if (s.d4 <= 128) TENSAIR_STEP(4);
    else TENSAIR_STEP(8);
#undef TENSAIR_STEP
    return cudaGetLastError();
}

// One warp per row: dot product and both squared norms in fp64, combined by shuffles.
__global__ void __launch_bounds__(256)
k_cosine_difference(const float* __restrict__ rows, const float* __restrict__ snap, float* __restrict__ out,
                    uint32_t nrows, uint32_t d, uint32_t stride) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    for (uint32_t r = warp; r < nrows; r += nwarps) {
        const float* a = rows + (size_t)r * stride;
        const float* b = snap + (size_t)r * d;
        double ab = 0.0, aa = 0.0, bb = 0.0;
        for (uint32_t e = lane; e < d; e += 32) {
            const double x = (double)a[e], y = (double)b[e];
            ab = fma(x, y, ab);
            aa = fma(x, x, aa);
            bb = fma(y, y, bb);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            ab += __shfl_xor_sync(0xFFFFFFFFu, ab, o);
            aa += __shfl_xor_sync(0xFFFFFFFFu, aa, o);
            bb += __shfl_xor_sync(0xFFFFFFFFu, bb, o);
        }
        if (lane == 0) {
            double diff;
            if (aa == 0.0 && bb == 0.0) diff = 0.0;
            else if (aa == 0.0 || bb == 0.0) diff = 1.0;
            else diff = 1.0 - ab / (sqrt(aa) * sqrt(bb));
            out[r] = (float)diff;
        }
    }
}

cudaError_t launch_cosine_difference(const Launcher& L, const float* rows, const float* snap, float* out, uint32_t nrows,
                                     const Shape& s) {
    if (!nrows) return cudaSuccess;
    uint32_t blocks = (nrows + 7) / 8;
    if (blocks > (uint32_t)L.sms * 32) blocks = (uint32_t)L.sms * 32;
    Timed timed(L, K_COSINE);
    k_cosine_difference<<<blocks, 256, 0, L.stream>>>(rows, snap, out, nrows, s.d, s.stride);
    return cudaGetLastError();
}

cudaError_t launch_apply(const Launcher& L, const MsgHeader* hdr, const uint32_t* ids, const float* delta,
                         float* table, const Shape& s) {
    return launch_apply_rows(L, hdr, ids, delta, table, s, 0);
}

}  // namespace tensair
