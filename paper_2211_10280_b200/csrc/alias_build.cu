// Device builder of the negative sampler's alias table (rebuilt when the stream drifts).  The table is
// defined in exact integers (see build_alias_host in sampler.cu for the definition), so this parallel
// construction from scans and binary searches gives the same bits as the sequential host builder:
//   weights and their maximum -> integer masses, their sum and the first largest entry -> capacity C ->
//   per-tile counts and sums of light deficits / heavy surpluses -> scan of the tiles -> rank, index and
//   running sum of every entry -> one thread per entry finds by binary search who tops its bucket up.
#include "kernels.h"

namespace tensair {

namespace {

constexpr int kTile = 1024;

struct TileSum { unsigned long long deficit, surplus; uint32_t lights, pad; };

__device__ inline unsigned long long warp_max(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = other > v ? other : v;
    }
    return v;
}
__device__ inline unsigned long long warp_sum(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

__global__ void k_alias_reset(AliasState* st) {
    st->heaviest_bits = 0;
    st->sum = 0;
    st->top = 0;
    st->first_top = ~0ull;
    st->lights = 0;
}

// weight = (sqrt(sqrt(count)))^3 in fp64 and the largest weight (positive doubles order like their bit patterns)
__global__ void __launch_bounds__(256)
k_alias_weight(const unsigned long long* __restrict__ counts, uint32_t V, double* __restrict__ weight, AliasState* st) {
    const uint32_t i = blockIdx.x * 256 + threadIdx.x;
    double w = 0.0;
    if (i < V) {
        const double root4 = sqrt(sqrt(__ull2double_rn(counts[i])));
        w = __dmul_rn(__dmul_rn(root4, root4), root4);
        weight[i] = w;
    }
    const unsigned long long m = warp_max((unsigned long long)__double_as_longlong(w));
    if ((threadIdx.x & 31) == 0 && m) atomicMax(&st->heaviest_bits, m);
}

// mass = floor(weight * 2^(bits - e)), 2^(e-1) <= largest weight < 2^e; in place over the weights
__global__ void __launch_bounds__(256)
k_alias_mass(unsigned long long* __restrict__ mass, uint32_t V, int bits, AliasState* st) {
    const uint32_t i = blockIdx.x * 256 + threadIdx.x;
    const int shift = bits - (ilogb(__longlong_as_double((long long)st->heaviest_bits)) + 1);
    unsigned long long m = 0;
    if (i < V) {
        m = __double2ull_rd(ldexp(__longlong_as_double((long long)mass[i]), shift));
        mass[i] = m;
    }
    const unsigned long long s = warp_sum(m), t = warp_max(m);
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(&st->sum, s);
        atomicMax(&st->top, t);
    }
}

__global__ void __launch_bounds__(256)
k_alias_first_top(const unsigned long long* __restrict__ mass, uint32_t V, AliasState* st) {
    const uint32_t i = blockIdx.x * 256 + threadIdx.x;
    if (i < V && mass[i] == st->top) atomicMin(&st->first_top, (unsigned long long)i);
}

__device__ inline unsigned long long capacity(const AliasState* st, uint32_t V) { return (st->sum + V - 1) / V; }

// Raises the first largest entry so that the masses add up to C * V, and sums every tile's lights.
__global__ void __launch_bounds__(kTile)
k_alias_tiles(unsigned long long* __restrict__ mass, uint32_t V, const AliasState* __restrict__ st, TileSum* __restrict__ tiles) {
    __shared__ unsigned long long s_def[32], s_sur[32];
    __shared__ uint32_t s_cnt[32];
    const unsigned long long cap = capacity(st, V);
    const uint32_t i = blockIdx.x * kTile + threadIdx.x;
    unsigned long long def = 0, sur = 0;
    uint32_t light = 0;
    if (i < V) {
        unsigned long long m = mass[i];
        if (i == st->first_top) {
            m += cap * V - st->sum;
            mass[i] = m;
        }
        if (m < cap) { light = 1; def = cap - m; } else sur = m - cap;
    }
    def = warp_sum(def);
    sur = warp_sum(sur);
    light = (uint32_t)warp_sum(light);
    const uint32_t w = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) { s_def[w] = def; s_sur[w] = sur; s_cnt[w] = light; }
    __syncthreads();
    if (w == 0) {
        def = warp_sum(s_def[threadIdx.x]);
        sur = warp_sum(s_sur[threadIdx.x]);
        light = (uint32_t)warp_sum(s_cnt[threadIdx.x]);
        if (threadIdx.x == 0) tiles[blockIdx.x] = TileSum{def, sur, light, 0u};
    }
}

// Exclusive scan over the tiles, in place, by one block; leaves the number of light entries in the state.
__global__ void __launch_bounds__(kTile)
k_alias_scan_tiles(TileSum* __restrict__ tiles, uint32_t n_tiles, AliasState* st) {
    __shared__ unsigned long long s_def[kTile], s_sur[kTile];
    __shared__ uint32_t s_cnt[kTile];
    unsigned long long carry_def = 0, carry_sur = 0;
    uint32_t carry_cnt = 0;
    for (uint32_t base = 0; base < n_tiles; base += kTile) {
        const uint32_t t = base + threadIdx.x;
        const TileSum mine = t < n_tiles ? tiles[t] : TileSum{0, 0, 0, 0};
        s_def[threadIdx.x] = mine.deficit; s_sur[threadIdx.x] = mine.surplus; s_cnt[threadIdx.x] = mine.lights;
        __syncthreads();
        for (int o = 1; o < kTile; o <<= 1) {      // inclusive scan of the chunk
            unsigned long long a = 0, b = 0;
            uint32_t c = 0;
            if ((int)threadIdx.x >= o) { a = s_def[threadIdx.x - o]; b = s_sur[threadIdx.x - o]; c = s_cnt[threadIdx.x - o]; }
            __syncthreads();
            s_def[threadIdx.x] += a; s_sur[threadIdx.x] += b; s_cnt[threadIdx.x] += c;
            __syncthreads();
        }
        if (t < n_tiles)
            tiles[t] = TileSum{carry_def + s_def[threadIdx.x] - mine.deficit, carry_sur + s_sur[threadIdx.x] - mine.surplus,
                               carry_cnt + s_cnt[threadIdx.x] - mine.lights, 0u};
        carry_def += s_def[kTile - 1]; carry_sur += s_sur[kTile - 1]; carry_cnt += s_cnt[kTile - 1];
        __syncthreads();
    }
    if (threadIdx.x == 0) st->lights = carry_cnt;
}

// Rank of every entry among the light (or heavy) ones, in index order, with the running sum up to and including it.
// Light rank n goes to position n, heavy rank t to position (number of lights) + t.
__global__ void __launch_bounds__(kTile)
k_alias_rank(const unsigned long long* __restrict__ mass, uint32_t V, const AliasState* __restrict__ st,
             const TileSum* __restrict__ tiles, uint32_t* __restrict__ rank_at, unsigned long long* __restrict__ run_sum) {
    __shared__ unsigned long long s_def[32], s_sur[32];
    __shared__ uint32_t s_cnt[32];
    const unsigned long long cap = capacity(st, V);
    const uint32_t i = blockIdx.x * kTile + threadIdx.x, lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    unsigned long long def = 0, sur = 0;
    uint32_t light = 0;
    const bool valid = i < V;
    unsigned long long m = 0;
    if (valid) {
        m = mass[i];
        if (m < cap) { light = 1; def = cap - m; } else sur = m - cap;
    }
    // inclusive scans inside the warp
    unsigned long long idef = def, isur = sur;
    uint32_t icnt = light;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long a = __shfl_up_sync(0xFFFFFFFFu, idef, o), b = __shfl_up_sync(0xFFFFFFFFu, isur, o);
        const uint32_t c = __shfl_up_sync(0xFFFFFFFFu, icnt, o);
        if ((int)lane >= o) { idef += a; isur += b; icnt += c; }
    }
    if (lane == 31) { s_def[w] = idef; s_sur[w] = isur; s_cnt[w] = icnt; }
    __syncthreads();
    if (w == 0) {                                 // exclusive scan of the 32 warp totals
        unsigned long long a = s_def[lane], b = s_sur[lane];
        uint32_t c = s_cnt[lane];
        const unsigned long long a0 = a, b0 = b;
        const uint32_t c0 = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long x = __shfl_up_sync(0xFFFFFFFFu, a, o), y = __shfl_up_sync(0xFFFFFFFFu, b, o);
            const uint32_t z = __shfl_up_sync(0xFFFFFFFFu, c, o);
            if ((int)lane >= o) { a += x; b += y; c += z; }
        }
        s_def[lane] = a - a0; s_sur[lane] = b - b0; s_cnt[lane] = c - c0;
    }
    __syncthreads();
    if (!valid) return;
    const TileSum before = tiles[blockIdx.x];
    const uint32_t lights_before = before.lights + s_cnt[w] + icnt - light;          // light entries with a smaller index
    if (light) {
        rank_at[lights_before] = i;
        run_sum[lights_before] = before.deficit + s_def[w] + idef;
    } else {
        const uint32_t at = st->lights + (i - lights_before);
        rank_at[at] = i;
        run_sum[at] = before.surplus + s_sur[w] + isur;
    }
}

__device__ inline uint32_t kept_to_thresh(unsigned long long kept, unsigned long long cap) {
    return (uint32_t)__double2ull_rd(__dmul_rn(__ddiv_rn(__ull2double_rn(kept), __ull2double_rn(cap)), 4294967296.0));
}

// One thread per rank position: who tops this entry's bucket up, and how much of it the entry keeps.
__global__ void __launch_bounds__(256)
k_alias_pair(const unsigned long long* __restrict__ mass, uint32_t V, const AliasState* __restrict__ st,
             const uint32_t* __restrict__ rank_at, const unsigned long long* __restrict__ run_sum, uint2* __restrict__ table) {
    const uint32_t r = blockIdx.x * 256 + threadIdx.x;
    if (r >= V) return;
    const unsigned long long cap = capacity(st, V);
    const uint32_t lights = st->lights, heavies = V - lights;
    const unsigned long long* deficit_sum = run_sum;            // [lights]
    const unsigned long long* surplus_sum = run_sum + lights;   // [heavies]
    const uint32_t i = rank_at[r];
    if (r < lights) {
        const unsigned long long m = mass[i];
        const unsigned long long before = deficit_sum[r] - (cap - m);
        uint32_t lo = 0, hi = heavies;                           // first t with surplus_sum[t] > before
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (surplus_sum[mid] > before) hi = mid; else lo = mid + 1;
        }
        table[i] = make_uint2(kept_to_thresh(m, cap), rank_at[lights + lo]);
        return;
    }
    const uint32_t t = r - lights;
    const unsigned long long given = surplus_sum[t];
    uint2 entry = make_uint2(0xFFFFFFFFu, i);
    if (t + 1 < heavies && given != 0) {
        uint32_t lo = 0, hi = lights;                            // first n with deficit_sum[n] >= given
        while (lo < hi) {
            const uint32_t mid = (lo + hi) >> 1;
            if (deficit_sum[mid] >= given) hi = mid; else lo = mid + 1;
        }
        const unsigned long long kept = cap + given - deficit_sum[lo];
        if (kept < cap) entry = make_uint2(kept_to_thresh(kept, cap), rank_at[r + 1]);
    }
    table[i] = entry;
}

}  // namespace

size_t alias_work_bytes(uint32_t V) {
    const size_t tiles = ((size_t)V + kTile - 1) / kTile;
    return (size_t)V * 8 + (size_t)V * 8 + (((size_t)V * 4 + 255) / 256) * 256 + tiles * sizeof(TileSum) + 256;
}

cudaError_t launch_alias_build(const Launcher& L, const unsigned long long* counts, uint32_t V, AliasState* st,
                               uint8_t* work, uint2* table) {
    const uint32_t tiles = (V + kTile - 1) / kTile;
    unsigned long long* mass = reinterpret_cast<unsigned long long*>(work);
    unsigned long long* run_sum = mass + V;
    uint32_t* rank_at = reinterpret_cast<uint32_t*>(run_sum + V);
    TileSum* tile_sums = reinterpret_cast<TileSum*>(work + (size_t)V * 16 + (((size_t)V * 4 + 255) / 256) * 256);
    const uint32_t blocks = (V + 255) / 256;
    { Timed timed(L, K_ALIAS_BUILD); k_alias_reset<<<1, 1, 0, L.stream>>>(st); }
    { Timed timed(L, K_ALIAS_BUILD); k_alias_weight<<<blocks, 256, 0, L.stream>>>(counts, V, reinterpret_cast<double*>(mass), st); }
    { Timed timed(L, K_ALIAS_BUILD); k_alias_mass<<<blocks, 256, 0, L.stream>>>(mass, V, alias_mass_bits(V), st); }
    { Timed timed(L, K_ALIAS_BUILD); k_alias_first_top<<<blocks, 256, 0, L.stream>>>(mass, V, st); }
    { Timed timed(L, K_ALIAS_BUILD); k_alias_tiles<<<tiles, kTile, 0, L.stream>>>(mass, V, st, tile_sums); }
    { Timed timed(L, K_ALIAS_BUILD); k_alias_scan_tiles<<<1, kTile, 0, L.stream>>>(tile_sums, tiles, st); }
    { Timed timed(L, K_ALIAS_BUILD); k_alias_rank<<<tiles, kTile, 0, L.stream>>>(mass, V, st, tile_sums, rank_at, run_sum); }
    { Timed timed(L, K_ALIAS_BUILD); k_alias_pair<<<blocks, 256, 0, L.stream>>>(mass, V, st, rank_at, run_sum, table); }
    return cudaGetLastError();
}

}  // namespace tensair
