// Sum of buffered gradient messages (Algorithm 1 with maxGradBuffer = m > 1: gradients are accumulated and sent
// after every m-th mini-batch).  The m messages of one replica are merged into one: the union of their
// rows, each row the fp32 sum of its delta rows in the order the messages were computed.
//
// Every message carries an index of its rows by ranges of 16 ids (buckets), so the merge works bucket by
// bucket: the ids of a bucket in message k form a 16-bit mask; the union mask gives the bucket's merged
// rows; an exclusive scan of the mask popcounts gives their positions - which is also the bucket index
// of the merged message.
#include "kernels.h"

namespace tensair {

__device__ inline uint32_t bucket_mask(const uint32_t* __restrict__ ids, uint32_t beg, uint32_t end) {
    uint32_t mask = 0;
    for (uint32_t m = beg; m < end; ++m) mask |= 1u << (__ldg(ids + m) & ((1u << kBucketShift) - 1));
    return mask;
}

// One thread per bucket: how many distinct rows the messages have there.
__global__ void __launch_bounds__(256)
k_merge_count(MergeInputs in, uint32_t n_buckets, uint32_t* __restrict__ counts) {
    const uint32_t b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= n_buckets) return;
    uint32_t mask = 0;
    for (uint32_t k = 0; k < in.count; ++k) mask |= bucket_mask(in.ids[k], __ldg(in.buckets[k] + b), __ldg(in.buckets[k] + b + 1));
    counts[b] = __popc(mask);
}

// One block: exclusive scan of the bucket counts into the merged message's bucket index; row count in the header.
__global__ void __launch_bounds__(1024)
k_merge_scan(const uint32_t* __restrict__ counts, uint32_t n_buckets, uint32_t* __restrict__ bucket_start,
             MsgHeader* __restrict__ hdr, uint32_t capacity, uint32_t* __restrict__ err) {
    __shared__ uint32_t warp_tot[32];
    __shared__ uint32_t carry_s;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (uint32_t base = 0; base < n_buckets; base += 1024) {
        const uint32_t idx = base + threadIdx.x;
        const uint32_t v = idx < n_buckets ? counts[idx] : 0;
        uint32_t incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= (uint32_t)o) incl += t;
        }
        if (lane == 31) warp_tot[wid] = incl;
        __syncthreads();
        if (wid == 0) {
            const uint32_t t = warp_tot[lane];
            uint32_t ti = t;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, ti, o);
                if (lane >= (uint32_t)o) ti += u;
            }
            warp_tot[lane] = ti - t;
        }
        __syncthreads();
        const uint32_t carry = carry_s;
        if (idx < n_buckets) bucket_start[idx] = carry + warp_tot[wid] + incl - v;
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = carry + warp_tot[wid] + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        bucket_start[n_buckets] = carry_s;
        // The slots are sized for the largest union there can be; should one still not fit, the message is cut
        // at the slot's capacity (the write kernel skips the rows past it) and the error word says so.
        if (carry_s > capacity) atomicOr(err, kErrOverflow);
        hdr->n_rows = carry_s < capacity ? carry_s : capacity;
        hdr->n_items = 0;
        hdr->pad = 0;
    }
}

// One warp per bucket: writes the merged ids and the summed delta rows of the bucket.
template <int NV>
__global__ void __launch_bounds__(128)
k_merge_write(MergeInputs in, uint32_t n_buckets, uint32_t V, const uint32_t* __restrict__ bucket_start,
              MsgHeader* __restrict__ hdr, uint32_t* __restrict__ out_ids, float4* __restrict__ out_delta, uint32_t d4,
              uint32_t stride4, uint32_t capacity) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    for (uint32_t b = warp; b < n_buckets; b += nwarps) {
        uint32_t beg[kMaxMerge], mask[kMaxMerge];
        uint32_t all = 0;
#pragma unroll
        for (int k = 0; k < kMaxMerge; ++k) {
            beg[k] = 0;
            mask[k] = 0;
            if ((uint32_t)k < in.count) {
                beg[k] = __ldg(in.buckets[k] + b);
                mask[k] = bucket_mask(in.ids[k], beg[k], __ldg(in.buckets[k] + b + 1));
                all |= mask[k];
            }
        }
        const uint32_t base = bucket_start[b];
        const uint32_t first_id = b << kBucketShift;
        // the first output row (id >= V) marks the end of the input rows
        if (lane == 0 && V >= first_id && V < first_id + (1u << kBucketShift))
            hdr->n_in_rows = min(base + __popc(all & ((1u << (V - first_id)) - 1)), capacity);
        uint32_t rest = all;
        while (rest) {
            const uint32_t j = __ffs(rest) - 1;
            rest &= rest - 1;
            const uint32_t below = (1u << j) - 1;
            const uint32_t pos = base + __popc(all & below);
            if (pos >= capacity) break;   // positions ascend with j: nothing further of this bucket fits either
            float4 acc[NV];
            bool have = false;
#pragma unroll
            for (int k = 0; k < kMaxMerge; ++k) {
                if ((uint32_t)k < in.count && (mask[k] >> j & 1u)) {
                    const float4* src = reinterpret_cast<const float4*>(in.delta[k]) +
                                        (size_t)(beg[k] + __popc(mask[k] & below)) * stride4;
#pragma unroll
                    for (int i = 0; i < NV; ++i) {
                        const uint32_t e = lane + 32 * i;
                        if (e < d4) {
                            const float4 x = __ldg(src + e);
                            if (!have) acc[i] = x;
                            else { acc[i].x += x.x; acc[i].y += x.y; acc[i].z += x.z; acc[i].w += x.w; }
                        }
                    }
                    have = true;
                }
            }
            if (lane == 0) out_ids[pos] = first_id + j;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const uint32_t e = lane + 32 * i;
                if (e < d4) out_delta[(size_t)pos * stride4 + e] = acc[i];
            }
        }
    }
}

cudaError_t launch_merge(const Launcher& L, const MergeInputs& in, MsgHeader* hdr, uint32_t* bucket_start, uint32_t* ids,
                         float* delta, uint32_t* counts, const Shape& s, uint32_t capacity, uint32_t* err) {
    const uint32_t nb = bucket_count(s.V);
    const uint32_t stride4 = s.stride / 4;
    float4* d4p = reinterpret_cast<float4*>(delta);
    {
        Timed timed(L, K_MERGE);
        k_merge_count<<<(nb + 255) / 256, 256, 0, L.stream>>>(in, nb, counts);
    }
    {
        Timed timed(L, K_MERGE);
        k_merge_scan<<<1, 1024, 0, L.stream>>>(counts, nb, bucket_start, hdr, capacity, err);
    }
    uint32_t blocks = (uint32_t)L.sms * 32;
    if (blocks > (nb + 3) / 4) blocks = (nb + 3) / 4;
    Timed timed(L, K_MERGE);
#define TENSAIR_MERGE(NV) \
    k_merge_write<NV><<<blocks, 128, 0, L.stream>>>(in, nb, s.V, bucket_start, hdr, ids, d4p, s.d4, stride4, capacity)
    if (s.d4 <= 32) TENSAIR_MERGE(1);
    else if (s.d4 <= 64) TENSAIR_MERGE(2);
    else if (s.d4 <= 96) TENSAIR_MERGE(3);
    else if (s.d4 <= 128) TENSAIR_MERGE(4);
    else TENSAIR_MERGE(8);
#undef TENSAIR_MERGE
    return cudaGetLastError();
}

}  // namespace tensair
