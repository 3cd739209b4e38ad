// The rows that drifted most (Section 4.3, Table 1 lists the words whose embeddings moved most): the k
// largest entries of an array of per-row cosine differences, largest first, the smaller row first among
// equal values.  Every entry gets a distinct 64-bit rank key (value in the total order of fp32 bit patterns,
// then the complement of the row index), the k-th largest key is found by an 8-pass radix select that
// only histograms the array, the k entries at or above it are collected, and one block sorts them.
#include "kernels.h"

namespace tensair {

namespace {

__device__ inline uint64_t rank_key(float x, uint32_t id) {
    const uint32_t b = __float_as_uint(x);
    const uint32_t ord = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
    return ((uint64_t)ord << 32) | (uint64_t)(0xFFFFFFFFu - id);
}

__global__ void k_topk_init(TopkState* st, uint32_t k) {
    st->hist[threadIdx.x] = 0;
    if (threadIdx.x == 0) {
        st->prefix = 0;
        st->remaining = k;
        st->n_out = 0;
    }
}

// Histogram of byte `pass` (0 = most significant) of the keys whose higher bytes equal the prefix found so far.
__global__ void __launch_bounds__(256)
k_topk_hist(const float* __restrict__ diff, uint32_t n, uint32_t pass, TopkState* __restrict__ st) {
    __shared__ uint32_t h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const uint64_t prefix = st->prefix;
    const uint32_t shift = 56 - 8 * pass;
    for (uint64_t i = (uint64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (uint64_t)gridDim.x * 256) {
        const uint64_t key = rank_key(diff[i], (uint32_t)i);
        if (pass == 0 || (key >> (shift + 8)) == prefix) atomicAdd(&h[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (h[threadIdx.x]) atomicAdd(&st->hist[threadIdx.x], h[threadIdx.x]);
}

// The byte of the k-th largest key: the largest digit D with (keys of a larger digit) < remaining.
__global__ void k_topk_pick(TopkState* st) {
    __shared__ uint32_t h[256];
    h[threadIdx.x] = st->hist[threadIdx.x];
    st->hist[threadIdx.x] = 0;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t above = 0, digit = 0;
        for (int dgt = 255; dgt >= 0; --dgt) {
            if (above + h[dgt] >= st->remaining) { digit = (uint32_t)dgt; break; }
            above += h[dgt];
        }
        st->remaining -= above;
        st->prefix = (st->prefix << 8) | digit;
    }
}

__global__ void __launch_bounds__(256)
k_topk_collect(const float* __restrict__ diff, uint32_t n, TopkState* __restrict__ st, uint32_t cap) {
    const uint64_t kth = st->prefix;
    for (uint64_t i = (uint64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (uint64_t)gridDim.x * 256) {
        const uint64_t key = rank_key(diff[i], (uint32_t)i);
        if (key >= kth) {
            const uint32_t slot = atomicAdd(&st->n_out, 1u);
            if (slot < cap) st->keys[slot] = key;
        }
    }
}

// Bitonic sort of the collected keys, descending, in one block; then the keys are taken apart again.
__global__ void __launch_bounds__(1024)
k_topk_sort(const TopkState* __restrict__ st, uint32_t k, uint32_t* __restrict__ ids, float* __restrict__ vals) {
    __shared__ uint64_t key[kTopkMax];
    uint32_t n2 = 1;
    while (n2 < k) n2 <<= 1;
    for (uint32_t i = threadIdx.x; i < n2; i += 1024) key[i] = i < k ? st->keys[i] : 0ull;
    __syncthreads();
    for (uint32_t size = 2; size <= n2; size <<= 1) {
        for (uint32_t stride = size >> 1; stride > 0; stride >>= 1) {
            for (uint32_t t = threadIdx.x; t < n2 / 2; t += 1024) {
                const uint32_t lo = 2 * t - (t & (stride - 1));
                const uint32_t hi = lo + stride;
                const bool descending = (lo & size) == 0;
                const uint64_t a = key[lo], b = key[hi];
                if ((a < b) == descending) { key[lo] = b; key[hi] = a; }
            }
            __syncthreads();
        }
    }
    for (uint32_t i = threadIdx.x; i < k; i += 1024) {
        const uint32_t ord = (uint32_t)(key[i] >> 32);
        const uint32_t b = (ord & 0x80000000u) ? (ord & 0x7FFFFFFFu) : ~ord;
        ids[i] = 0xFFFFFFFFu - (uint32_t)key[i];
        vals[i] = __uint_as_float(b);
    }
}

}  // namespace

cudaError_t launch_top_drifted(const Launcher& L, const float* diff, uint32_t n, uint32_t k, TopkState* st,
                               uint32_t* ids, float* vals) {
    if (k == 0 || n == 0) return cudaSuccess;
    uint32_t blocks = (n + 255) / 256;
    const uint32_t most = (uint32_t)L.sms * 8;
    if (blocks > most) blocks = most;
    {
        Timed timed(L, K_TOPK);
        k_topk_init<<<1, 256, 0, L.stream>>>(st, k);
    }
    for (uint32_t pass = 0; pass < 8; ++pass) {
        {
            Timed timed(L, K_TOPK);
            k_topk_hist<<<blocks, 256, 0, L.stream>>>(diff, n, pass, st);
        }
        Timed timed(L, K_TOPK);
        k_topk_pick<<<1, 256, 0, L.stream>>>(st);
    }
    {
        Timed timed(L, K_TOPK);
        k_topk_collect<<<blocks, 256, 0, L.stream>>>(diff, n, st, kTopkMax);
    }
    Timed timed(L, K_TOPK);
    k_topk_sort<<<1, 1024, 0, L.stream>>>(st, k, ids, vals);
    return cudaGetLastError();
}

}  // namespace tensair
