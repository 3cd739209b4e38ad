// Stable least-significant-digit radix sort of 64-bit items by (a bit range of) their 32-bit keys.
//
// Keys are row ids, dense in [0, 2V], so few digit passes are needed.  Every pass is three kernels:
// per-tile digit histogram, per-digit scan over the tiles (one warp per digit), stable scatter; with few tiles
// the scan is left out and every scatter block sums the tile counts it needs itself.  Stability
// (equal keys keep their input order) is what makes the later per-row sums run in a fixed order.
// The whole working set (two item buffers) stays in L2 at the sizes of interest.
#include "kernels.h"

namespace tensair {

constexpr int kRadixBits = 8;
constexpr int kBins = 1 << kRadixBits;
constexpr int kSortThreads = 256;
constexpr int kSortWarps = kSortThreads / 32;
constexpr int kItemsPerThread = 16;
constexpr int kTile = kSortThreads * kItemsPerThread;   // 4096 items per block
constexpr int kWarpSpan = 32 * kItemsPerThread;         // consecutive items owned by one warp

uint32_t sort_tiles(uint32_t n) { return (n + kTile - 1) / kTile; }
uint32_t sort_hist_words(uint32_t n) { return (sort_tiles(n) + 1) * kBins; }   // per-tile counts, then digit totals

__global__ void __launch_bounds__(kSortThreads)
k_radix_hist(const item_t* __restrict__ in, uint32_t n, uint32_t shift, uint32_t* __restrict__ hist, uint32_t tiles) {
    __shared__ uint32_t h[kBins];
    h[threadIdx.x] = 0;
    __syncthreads();
    const uint32_t base = blockIdx.x * kTile;
#pragma unroll 4
    for (int i = 0; i < kItemsPerThread; ++i) {
        const uint32_t idx = base + i * kSortThreads + threadIdx.x;
        if (idx < n) atomicAdd(&h[(item_key(in[idx]) >> shift) & (kBins - 1)], 1u);
    }
    __syncthreads();
    hist[threadIdx.x * tiles + blockIdx.x] = h[threadIdx.x];   // digit-major
}

// Per digit: exclusive scan, in place, of its per-tile counts (one warp per digit), and the digit's total.
constexpr int kScanWarps = 8;
__global__ void __launch_bounds__(kScanWarps * 32)
k_scan_digits(uint32_t* __restrict__ hist, uint32_t tiles, uint32_t* __restrict__ totals) {
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t digit = blockIdx.x * kScanWarps + (threadIdx.x >> 5);
    uint32_t* row = hist + (size_t)digit * tiles;
    uint32_t carry = 0;
    for (uint32_t base = 0; base < tiles; base += 32) {
        const uint32_t idx = base + lane;
        const uint32_t v = idx < tiles ? row[idx] : 0;
        uint32_t incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= (uint32_t)o) incl += t;
        }
        if (idx < tiles) row[idx] = carry + incl - v;
        carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
    if (lane == 0) totals[digit] = carry;
}

// Stable scatter.  Warp w of a block owns the consecutive items [w*512, (w+1)*512) of the tile and
// walks them 32 at a time; lanes with the same digit are ranked by lane order within a round and
// rounds are ranked by their order, so the rank of an item among equal digits follows input order.
// At most 64 registers per thread: a block of 256 threads then needs 16 K registers of a multiprocessor, which the
// forward kernel, beside which the sort runs, leaves free when it sizes its grid.
// kRawHist: `hist` holds the per-tile counts as the histogram kernel left them (no scan kernel ran): every block adds
// up, per digit, the tiles before it and all tiles itself - cheaper than a launch when there are few tiles.
constexpr uint32_t kMaxRawTiles = 32;   // measured: at 81 tiles the scan kernel is the cheaper way again
template <bool kRawHist>
__global__ void __launch_bounds__(kSortThreads, 4)
k_radix_scatter(const item_t* __restrict__ in, item_t* __restrict__ out, uint32_t n, uint32_t shift,
                const uint32_t* __restrict__ hist, uint32_t tiles, const uint32_t* __restrict__ totals, Limits lim) {
    __shared__ uint32_t cnt[kSortWarps][kBins];
    __shared__ uint32_t digit_base[kBins];
    __shared__ uint32_t warp_tot[kSortWarps];
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < kSortWarps * kBins; i += kSortThreads) (&cnt[0][0])[i] = 0;
    __syncthreads();
    item_t item[kItemsPerThread];
    uint32_t rank[kItemsPerThread];
    const uint32_t wbase = blockIdx.x * kTile + wid * kWarpSpan;
    const uint32_t lt_mask = (1u << lane) - 1;
#pragma unroll
    for (int r = 0; r < kItemsPerThread; ++r) {
        const uint32_t idx = wbase + r * 32 + lane;
        const bool valid = idx < n;
        item[r] = valid ? in[idx] : 0;
        const uint32_t live = __ballot_sync(0xFFFFFFFFu, valid);
        rank[r] = 0;
        if (valid) {
            const uint32_t digit = (item_key(item[r]) >> shift) & (kBins - 1);
            const uint32_t peers = __match_any_sync(live, digit);
            const int leader = __ffs(peers) - 1;
            uint32_t before = 0;
            if ((int)lane == leader) {
                before = cnt[wid][digit];
                cnt[wid][digit] = before + __popc(peers);
            }
            before = __shfl_sync(peers, before, leader);
            rank[r] = before + __popc(peers & lt_mask);
        }
        __syncwarp();
    }
    __syncthreads();
    // this tile's offset inside its digit's run, and the digit's total
    uint32_t tile_offset, t;
    if (kRawHist) {
        tile_offset = 0;
        t = 0;
        for (uint32_t x = 0; x < tiles; ++x) {
            const uint32_t c = hist[threadIdx.x * tiles + x];
            if (x < blockIdx.x) tile_offset += c;
            t += c;
        }
    } else {
        tile_offset = hist[threadIdx.x * tiles + blockIdx.x];
        t = totals[threadIdx.x];
    }
    // exclusive scan of the digit totals: where each digit's run starts in the output
    {
        uint32_t incl = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t u = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= (uint32_t)o) incl += u;
        }
        if (lane == 31) warp_tot[wid] = incl;
        __syncthreads();
        uint32_t before = 0;
        for (uint32_t x = 0; x < wid; ++x) before += warp_tot[x];
        digit_base[threadIdx.x] = before + incl - t;
    }
    // per digit: start of the digit, this tile's offset in it, then exclusive prefix over the warps of the block
    {
        const uint32_t digit = threadIdx.x;
        uint32_t run = digit_base[digit] + tile_offset;
#pragma unroll
        for (int w = 0; w < kSortWarps; ++w) {
            const uint32_t c = cnt[w][digit];
            cnt[w][digit] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kItemsPerThread; ++r) {
        const uint32_t idx = wbase + r * 32 + lane;
        if (idx < n) {
            const uint32_t digit = (item_key(item[r]) >> shift) & (kBins - 1);
            const uint32_t pos = cnt[wid][digit] + rank[r];
            if (in_bounds(lim, pos, n)) out[pos] = item[r];
        }
    }
}

cudaError_t launch_sort(const Launcher& L, item_t* a, item_t* b, uint32_t n, uint32_t key_bits, uint32_t* hist,
                        item_t** sorted) {
    *sorted = a;
    if (n == 0) return cudaSuccess;
    const uint32_t tiles = sort_tiles(n);
    item_t* src = a;
    item_t* dst = b;
    for (uint32_t shift = 0; shift < key_bits; shift += kRadixBits) {
        {
            Timed timed(L, K_SORT_HIST);
            k_radix_hist<<<tiles, kSortThreads, 0, L.stream>>>(src, n, shift, hist, tiles);
        }
        if (tiles > kMaxRawTiles) {
            Timed timed(L, K_SORT_SCAN);
            k_scan_digits<<<kBins / kScanWarps, kScanWarps * 32, 0, L.stream>>>(hist, tiles, hist + (size_t)tiles * kBins);
        }
        {
            Timed timed(L, K_SORT_SCATTER);
            if (tiles > kMaxRawTiles)
                k_radix_scatter<false><<<tiles, kSortThreads, 0, L.stream>>>(src, dst, n, shift, hist, tiles, hist + (size_t)tiles * kBins, L.lim);
            else
                k_radix_scatter<true><<<tiles, kSortThreads, 0, L.stream>>>(src, dst, n, shift, hist, tiles, hist + (size_t)tiles * kBins, L.lim);
        }
        item_t* t = src; src = dst; dst = t;
    }
    *sorted = src;
    return cudaGetLastError();
}

}  // namespace tensair
