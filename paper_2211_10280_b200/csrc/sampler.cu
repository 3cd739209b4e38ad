// Negative sampler: alias table over count^0.75 (host build), token validation, and the kernel that
// draws the negatives of a batch and emits the sort items of all its contributions.
#include <algorithm>
#include <cmath>
#include <vector>

#include "kernels.h"
#include "philox.cuh"

namespace tensair {

// Walker alias table over weights count^0.75 in exact integer arithmetic, so that this host builder and the
// parallel device builder (alias_build.cu) give the same bits whatever order they work in.
//   weight = (sqrt(sqrt(count)))^3 in fp64 (only correctly rounded operations);
//   u = floor(weight * 2^(bits - e)) with 2^(e-1) <= largest weight < 2^e and bits = min(42, 62 - ceil(log2 V));
//   C = ceil(sum u / V), the first entry of largest u is raised so that sum u = C * V: V buckets of capacity C.
// Entries with u < C are light (deficit C - u), the others heavy (surplus u - C), each kind ranked in index
// order, with running sums D over the deficits and S over the surpluses.  Heavy entries give their mass
// away in rank order, to the light buckets in rank order and then to the bucket of the heavy entry before
// them; in terms of the sums: light n is topped up by the first heavy t with S_t > D_{n-1}; heavy t keeps
// C + S_t - D_n of its own bucket, n the first rank with D_n >= S_t, the rest comes from heavy t + 1.
// A bucket that keeps all of C accepts always (thresh 2^32-1, alias = self), otherwise
// thresh = floor(kept / C * 2^32), the quotient in fp64 from two exact operands.
int alias_mass_bits(uint32_t V) {
    int log2V = 0;
    while ((1ull << log2V) < V) ++log2V;
    return 62 - log2V < 42 ? 62 - log2V : 42;
}

void build_alias_host(const uint64_t* counts, uint32_t V, uint32_t* thresh, uint32_t* alias) {
    std::vector<double> weight(V);
    double heaviest = 0.0;
    for (uint32_t i = 0; i < V; ++i) {
        const double root4 = std::sqrt(std::sqrt(counts ? (double)counts[i] : 1.0));
        weight[i] = root4 * root4 * root4;
        heaviest = std::max(heaviest, weight[i]);
    }
    const int shift = alias_mass_bits(V) - (std::ilogb(heaviest) + 1);
    std::vector<uint64_t> mass(V);
    uint64_t sum = 0, top = 0;
    for (uint32_t i = 0; i < V; ++i) {
        mass[i] = (uint64_t)std::floor(std::ldexp(weight[i], shift));
        sum += mass[i];
        top = std::max(top, mass[i]);
    }
    const uint64_t cap = (sum + V - 1) / V;
    *std::find(mass.begin(), mass.end(), top) += cap * V - sum;

    std::vector<uint32_t> light_at, heavy_at;        // rank -> index
    std::vector<uint64_t> deficit_sum, surplus_sum;  // inclusive running sums by rank
    for (uint32_t i = 0; i < V; ++i) {
        if (mass[i] < cap) {
            light_at.push_back(i);
            deficit_sum.push_back((deficit_sum.empty() ? 0 : deficit_sum.back()) + (cap - mass[i]));
        } else {
            heavy_at.push_back(i);
            surplus_sum.push_back((surplus_sum.empty() ? 0 : surplus_sum.back()) + (mass[i] - cap));
        }
        thresh[i] = 0xFFFFFFFFu;
        alias[i] = i;
    }
    auto to_thresh = [cap](uint64_t kept) { return (uint32_t)std::floor((double)kept / (double)cap * 4294967296.0); };
    for (size_t n = 0; n < light_at.size(); ++n) {
        const uint32_t i = light_at[n];
        const uint64_t before = deficit_sum[n] - (cap - mass[i]);
        const size_t t = std::upper_bound(surplus_sum.begin(), surplus_sum.end(), before) - surplus_sum.begin();
        thresh[i] = to_thresh(mass[i]);
        alias[i] = heavy_at[t];
    }
    for (size_t t = 0; t + 1 < heavy_at.size(); ++t) {
        const uint64_t given = surplus_sum[t];
        if (given == 0) continue;                    // nothing to give: its bucket is its own
        const size_t n = std::lower_bound(deficit_sum.begin(), deficit_sum.end(), given) - deficit_sum.begin();
        const uint64_t kept = cap + given - deficit_sum[n];
        if (kept < cap) {
            thresh[heavy_at[t]] = to_thresh(kept);
            alias[heavy_at[t]] = heavy_at[t + 1];
        }
    }
}

// Checks the token ids; for a routed batch (owner != nullptr) also marks the centre positions whose word the
// hash partitioner gives to this replica, route(x) = mulhi32(Philox(x, 0, 0, route tag; seed).word0, W), and
// lists them (in no particular order: nothing downstream depends on it) so that the forward kernel can spread
// them evenly over its warps.
__global__ void k_validate(const int32_t* __restrict__ tok, uint32_t n, uint32_t V, uint32_t* err, uint8_t* owner,
                           uint32_t* __restrict__ owned, uint32_t* __restrict__ n_owned, uint32_t W, uint32_t replica,
                           uint32_t key0, uint32_t key1) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) {
        const int32_t t = tok[i];
        if (t < 0 || (uint32_t)t >= V) atomicOr(err, kErrBadToken);
        if (owner) {
            const Philox4 r = philox4x32_10(Philox4{(uint32_t)t, 0u, 0u, kTagRoute}, key0, key1);
            const bool mine = __umulhi(r.x, W) == replica;
            owner[i] = mine ? 1 : 0;
            if (mine) owned[atomicAdd(n_owned, 1u)] = i;
        }
    }
}

cudaError_t launch_validate(const Launcher& L, const int32_t* tok, uint32_t n, uint32_t V, uint32_t* err, uint8_t* owner,
                            uint32_t* owned, uint32_t* n_owned, uint32_t W, uint32_t replica, uint64_t seed) {
    if (n == 0) return cudaSuccess;
    if (owner) {
        const cudaError_t e = cudaMemsetAsync(n_owned, 0, 4, L.stream);
        if (e != cudaSuccess) return e;
    }
    Timed timed(L, K_VALIDATE);
    k_validate<<<(n + 255) / 256, 256, 0, L.stream>>>(tok, n, V, err, owner, owned, n_owned, W, replica, (uint32_t)seed,
                                                      (uint32_t)(seed >> 32));
    return cudaGetLastError();
}

__device__ inline uint32_t alias_pick(const uint2* __restrict__ tab, uint32_t V, uint32_t ra, uint32_t rb) {
    const uint32_t slot = __umulhi(ra, V);
    const uint2 e = __ldg(tab + slot);   // x = thresh, y = alias
    return (e.x == 0xFFFFFFFFu || rb < e.x) ? slot : e.y;
}

// One thread per (centre position q, window slot s, draw pair jp).  Window slot s in [0, 2w) stands
// for context position q + (s < w ? s - w : s - w + 1); slots outside the batch do nothing.
// Thread jp = 0 also emits the positive contribution; thread (s = 0, jp = 0) checks the position's token id (when
// `check` is set: the unrouted path has no separate validation kernel), counts the token (when `count` is set: only
// batches too short to have pairs are counted here, the others once the whole batch is known to be valid, by the
// first kernel of the message build) and emits the position's two input-row items: the forward kernel leaves one partial centre gradient for the pairs
// to the left of the position and one for those to its right (items 2q and 2q + 1; the contributions
// follow from item 2n on).  In a routed batch (owner != nullptr) the positions of other
// replicas' centre words emit only items that sort past every row and are never read.
__global__ void k_prepare(const int32_t* __restrict__ tok, uint32_t n, uint32_t V, uint32_t w, uint32_t k,
                          uint32_t replica, uint32_t batch_lo, uint32_t key0, uint32_t key1,
                          const uint2* __restrict__ alias_tab, uint32_t* __restrict__ rows,
                          item_t* __restrict__ items, unsigned long long* __restrict__ counts,
                          uint32_t* __restrict__ err, const uint8_t* __restrict__ owner, int check, int count, Limits lim) {
    if (*err) return;
    const uint32_t JP = (k + 1) / 2;
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint64_t total = (uint64_t)n * 2 * w * JP;
    if (t >= total) return;
    const uint32_t jp = (uint32_t)(t % JP);
    const uint32_t ps = (uint32_t)(t / JP);
    const uint32_t s = ps % (2 * w);
    const uint32_t q = ps / (2 * w);
    const uint32_t centre = (uint32_t)tok[q];
    const bool own = !owner || owner[q];
    if (s == 0 && jp == 0) {
        // A bad id only raises the flag here: nothing below indexes memory by a token id (row ids are stored, keys are
        // sorted by their low bits), and every later kernel of the batch sees the flag and leaves.
        if (check && centre >= V) atomicOr(err, kErrBadToken);
        if (count && own && centre < V) atomicAdd(counts + centre, 1ULL);
        if (n >= 2 && in_bounds(lim, 2ull * q + 1, lim.items)) {
            items[2 * q] = make_item(own ? centre : 2 * V, 2 * q);
            items[2 * q + 1] = make_item(own ? centre : 2 * V, 2 * q + 1);
        }
    }
    const int64_t c = (int64_t)q + (s < w ? (int64_t)s - (int64_t)w : (int64_t)s - (int64_t)w + 1);
    if (c < 0 || c >= (int64_t)n) return;
    const uint32_t lo = q > w ? q - w : 0;
    const uint32_t p = pair_offset(q, n, w) + ((uint32_t)c - lo) - ((uint32_t)c > q ? 1u : 0u);
    const uint32_t K1 = k + 1;
    const uint32_t ctx = (uint32_t)tok[c];
    const uint32_t cbase = p * K1;
    if (!in_bounds(lim, (uint64_t)cbase + K1 - 1, lim.contrib) || !in_bounds(lim, 2ull * n + cbase + K1 - 1, lim.items)) return;
    if (!own) {
        if (jp == 0) items[2 * n + cbase] = make_item(2 * V, cbase);
        const uint32_t j0 = 2 * jp;
        items[2 * n + cbase + 1 + j0] = make_item(2 * V, cbase + 1 + j0);
        if (j0 + 1 < k) items[2 * n + cbase + 2 + j0] = make_item(2 * V, cbase + 2 + j0);
        return;
    }
    if (jp == 0) {
        rows[cbase] = ctx;
        items[2 * n + cbase] = make_item(V + ctx, cbase);
    }
    const Philox4 r = philox4x32_10(Philox4{p, jp, batch_lo, kTagNegative | replica}, key0, key1);
    const uint32_t j0 = 2 * jp;
    const uint32_t n0 = alias_pick(alias_tab, V, r.x, r.y);
    rows[cbase + 1 + j0] = n0;
    items[2 * n + cbase + 1 + j0] = make_item(n0 == ctx ? 2 * V : V + n0, cbase + 1 + j0);
    if (j0 + 1 < k) {
        const uint32_t n1 = alias_pick(alias_tab, V, r.z, r.w);
        rows[cbase + 2 + j0] = n1;
        items[2 * n + cbase + 2 + j0] = make_item(n1 == ctx ? 2 * V : V + n1, cbase + 2 + j0);
    }
}

cudaError_t launch_prepare(const Launcher& L, const int32_t* tok, uint32_t n, const Shape& s, uint32_t replica,
                           uint32_t batch_lo, uint64_t seed, const uint2* alias_tab, uint32_t* rows,
                           item_t* items, unsigned long long* counts, uint32_t* err, const uint8_t* owner, bool check,
                           bool count) {
    if (n == 0) return cudaSuccess;
    const uint64_t total = (uint64_t)n * 2 * s.w * ((s.k + 1) / 2);
    const uint32_t blocks = (uint32_t)((total + 255) / 256);
    Timed timed(L, K_PREPARE);
    k_prepare<<<blocks, 256, 0, L.stream>>>(tok, n, s.V, s.w, s.k, replica, batch_lo, (uint32_t)seed,
                                            (uint32_t)(seed >> 32), alias_tab, rows, items, counts, err, owner, check ? 1 : 0,
                                            count ? 1 : 0, L.lim);
    return cudaGetLastError();
}

// Seeded initial input rows: U(-0.5/d, 0.5/d).  The 24 high bits of a Philox word, centred, give a
// uniform in (0,1) exactly representable in fp64; the division by d is taken in fp64, then rounded.
__global__ void k_init_input(float* __restrict__ table, uint32_t V, uint32_t d, uint32_t stride, uint32_t key0,
                             uint32_t key1) {
    const uint64_t blk = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;   // group of 4 consecutive elements
    const uint64_t total = (uint64_t)V * d;
    if (blk * 4 >= total) return;
    const Philox4 r = philox4x32_10(Philox4{(uint32_t)blk, (uint32_t)(blk >> 32), 0u, kTagInit}, key0, key1);
    const uint32_t words[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint64_t e = blk * 4 + i;
        if (e < total) {
            const double u = ((double)(words[i] >> 8) + 0.5) * (1.0 / 16777216.0);
            table[(e / d) * stride + (e % d)] = (float)((u - 0.5) / (double)d);
        }
    }
}

cudaError_t launch_init_input_table(const Launcher& L, float* table, const Shape& s, uint64_t seed) {
    const uint64_t groups = ((uint64_t)s.V * s.d + 3) / 4;
    Timed timed(L, K_INIT_TABLE);
    k_init_input<<<(uint32_t)((groups + 255) / 256), 256, 0, L.stream>>>(table, s.V, s.d, s.stride, (uint32_t)seed,
                                                                          (uint32_t)(seed >> 32));
    return cudaGetLastError();
}

}  // namespace tensair
