// Gradient calculation at the snapshot: fused gather -> dot -> sigmoid -> gradient scalars, centre-stationary.
// Rows are fp32 in memory; the dot products, the sigmoid and the partial sums are taken in fp64.
// Each output row is fetched from memory once per contribution (by a bulk asynchronous copy into
// shared memory) and serves both its dot product and the centre's gradient; the gradient scalar g
// (sigma(x) - 1 for the positive, sigma(x) for a negative, 0 for a negative equal to the positive) is
// recorded for the later per-output-row sums.
#include "kernels.h"

namespace tensair {


// ---- asynchronous bulk copies (global -> shared) completed on an mbarrier -------------------------
__device__ inline uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ inline void mbar_init(uint64_t* bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ inline void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ inline bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(smem_addr(bar)), "r"(parity) : "memory");
    return done != 0;
}
// Waits for a phase of the barrier, giving up after about a second.
__device__ inline bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > 2000000000LL) return false;
    return true;
}
__device__ inline void bulk_copy_g2s(void* dst_smem, const void* src_global, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst_smem)), "l"(src_global), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
// Orders this thread's earlier shared-memory reads before later asynchronous writes to the same memory.
__device__ inline void fence_generic_to_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// sigmoid(x) and -log(sigmoid(y)) for y = x or -x from one exponential e = exp(-|x|):
//   sigmoid(x) = 1 / (1 + e) for x >= 0, e / (1 + e) for x < 0;   -log(sigmoid(y)) = max(-y, 0) + log1p(e).
struct SigmoidLoss {
    double sig, softplus;   // sigmoid(x); log1p(exp(-|x|))
};
__device__ inline SigmoidLoss sigmoid_loss(double x) {
    const double e = exp(-fabs(x));
    const double r = 1.0 / (1.0 + e);
    return SigmoidLoss{x < 0.0 ? e * r : r, log1p(e)};
}

constexpr int kFwdWarps = 2;       // warps per block
// The radix sort of a batch runs on a second stream beside this kernel; its scatter kernel needs 256 threads x 64
// registers on a multiprocessor to get in at all.  The forward grid leaves that many registers free: measured
// with 120 registers per thread, 8 resident blocks (no room: the sort ends up behind the forward kernel) 5.79 ms
// per step, 6 blocks (room for one sort block) 5.57 ms although the forward kernel itself takes 0.40 instead of 0.31 ms.
constexpr int kRegistersLeftForTheSort = 256 * 64;

// A slice of VW consecutive floats of a row (VW = 4: one 16-byte load, VW = 2: one 8-byte load).
template <int VW> struct Slice;
template <> struct Slice<4> {
    static __device__ inline void load(const float* p, float (&a)[4]) {
        const float4 t = *reinterpret_cast<const float4*>(p);
        a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
    }
    static __device__ inline void load_global(const float* p, float (&a)[4]) {
        const float4 t = __ldg(reinterpret_cast<const float4*>(p));
        a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
    }
};
template <> struct Slice<2> {
    static __device__ inline void load(const float* p, float (&a)[2]) {
        const float2 t = *reinterpret_cast<const float2*>(p);
        a[0] = t.x; a[1] = t.y;
    }
    static __device__ inline void load_global(const float* p, float (&a)[2]) {
        const float2 t = __ldg(reinterpret_cast<const float2*>(p));
        a[0] = t.x; a[1] = t.y;
    }
};

// One warp per side of a centre position (grid-stride), no block-level cooperation.  For every pair of
// its side the warp stages the pair's 1 + k output rows into its own shared-memory buffer with one
// bulk asynchronous copy per row (all in flight together, completion counted by an mbarrier), then
//   1. takes the partial dot products of all staged rows with the centre row held in registers,
//   2. reduces them with a transposing shuffle network that leaves row j's dot product in lanes 2j, 2j+1,
//   3. evaluates sigmoid and loss for all rows at once (one row per lane pair instead of one per warp),
//   4. re-reads the staged rows and adds g * u to the centre gradient kept in registers.
// The partial centre gradient of the side is written once; nothing is shared between warps.
// A lane holds NV slices of VW floats of a row: slice lane + 32 * i.  VW is 4 unless 2 leaves fewer lanes idle
// (d = 300: 75 slices of 4 take three rounds of 32 lanes, 150 slices of 2 take five rounds of half the width).
// CR: rows reduced together (a power of two); 32 / CR lanes share a row's scalar.
// NR <= CR: rows of a whole chunk (the loops without predicates run over exactly NR staged rows).
template <int NV, int CR, int NR, int VW>
__global__ void __launch_bounds__(kFwdWarps * 32)
k_forward(const int32_t* __restrict__ tok, uint32_t n, uint32_t V, uint32_t d, uint32_t stride, uint32_t w,
          uint32_t k, uint32_t chunk_rows, uint32_t warp_stage, const float* __restrict__ table, const uint32_t* __restrict__ rows,
          Rec* __restrict__ rec, double* __restrict__ gin_pos, double* __restrict__ loss_pos, uint32_t* __restrict__ err,
          const uint32_t* __restrict__ owned, const uint32_t* __restrict__ n_owned, const uint32_t* __restrict__ batch_err,
          Limits lim) {
    // A batch prepared ahead of its turn raised its own error word (a later batch must not stop an earlier one that is
    // still at work); this, the batch's first kernel on the caller's stream, hands it on to the sticky word.
    if (batch_err && *batch_err) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(err, *batch_err);
        return;
    }
    if (*err) return;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint32_t lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    // warp_stage floats per warp: chunk_rows rows plus padding, so that slice lane + 32 * i (i < NV) of every
    // staged row is inside the buffer whatever the lane
    float* stage = reinterpret_cast<float*>(smem_raw) + (size_t)wib * warp_stage;
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem_raw + (size_t)kFwdWarps * warp_stage * sizeof(float)) + wib;
    if (lane == 0) mbar_init(bar, 1);
    __syncwarp();
    uint32_t parity = 0;
    bool failed = false;
    const uint32_t K1 = k + 1;
    const uint32_t row_bytes = d * 4;
    const uint32_t dv = d / VW;                               // slices of a row
    const float* __restrict__ tout = table + (size_t)V * stride;
    const uint32_t warp = blockIdx.x * kFwdWarps + wib, nwarps = gridDim.x * kFwdWarps;

    // A unit of work is one side of a centre position: the pairs with the context to its left, or to its
    // right (half a position's work, so that the units spread evenly over the warps).
    // routed batch: only the listed centre positions are this replica's
    const uint32_t n_units = 2 * (owned ? *n_owned : n);
    for (uint32_t at = warp; at < n_units && !failed; at += nwarps) {
        const uint32_t q = owned ? owned[at >> 1] : (at >> 1);
        const uint32_t side = at & 1u;
        const uint32_t centre = (uint32_t)tok[q];
        const float* __restrict__ vin = table + (size_t)centre * stride;
        double v[NV][VW], acc[NV][VW];
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const uint32_t e = lane + 32 * i;
            float f[VW];
#pragma unroll
            for (int c = 0; c < VW; ++c) f[c] = 0.f;
            if (e < dv) Slice<VW>::load_global(vin + e * VW, f);
            // the centre row carries the factor 2^896 that the staged rows lack (widen_down)
#pragma unroll
            for (int c = 0; c < VW; ++c) { v[i][c] = (double)f[c] * kWidenUp; acc[i][c] = 0.0; }
        }
        double loss = 0.0;
        const uint32_t lo = q > w ? q - w : 0;
        const uint32_t hi = q + w < n ? q + w : n - 1;
        const uint32_t c_beg = side ? q + 1 : lo, c_end = side ? hi + 1 : q;
        uint32_t p = pair_offset(q, n, w) + (side ? q - lo : 0u);
        // Row ids of a pair (lane l holds row l when a pair has at most 32 rows) and its context token are fetched
        // one pair ahead, so that a chunk's copies do not wait for a load of their addresses first.
        const bool ids_in_lanes = K1 <= 32;
        uint32_t ids_next = ids_in_lanes && lane < K1 && c_beg < c_end ? __ldg(rows + p * K1 + lane) : 0u;
        uint32_t ctx_next = c_beg < c_end ? (uint32_t)tok[c_beg] : 0u;
        for (uint32_t c = c_beg; c < c_end && !failed; ++c) {
            const uint32_t ctx = ctx_next, ids_pair = ids_next;
            const uint32_t cbase = p * K1;
            ++p;
            if (c + 1 < c_end) {
                if (ids_in_lanes && lane < K1) ids_next = __ldg(rows + p * K1 + lane);
                ctx_next = (uint32_t)tok[c + 1];
            }
            for (uint32_t j0 = 0; j0 < K1 && !failed; j0 += chunk_rows) {
                const uint32_t nr = K1 - j0 < chunk_rows ? K1 - j0 : chunk_rows;
                uint32_t rid = __shfl_sync(0xFFFFFFFFu, ids_pair, (j0 + lane) & 31u);
                if (!ids_in_lanes) rid = lane < nr ? __ldg(rows + cbase + j0 + lane) : 0u;
                const bool mine = lane < nr && (j0 + lane == 0 || rid != ctx) && in_bounds(lim, rid, V);
                const uint32_t live = __ballot_sync(0xFFFFFFFFu, mine);
                // stage the live rows: the buffer was last read by this warp, so order those reads first
                fence_generic_to_async();
                __syncwarp();
                if (lane == 0) mbar_arrive_expect_tx(bar, __popc(live) * row_bytes);
                __syncwarp();
                if (mine) bulk_copy_g2s(stage + (size_t)lane * stride, tout + (size_t)rid * stride, row_bytes, bar);
                if (__any_sync(0xFFFFFFFFu, !mbar_wait_bounded(bar, parity))) {
                    failed = true;
                    mbar_wait_bounded(bar, parity);   // give copies still in flight one more chance to land
                    break;
                }
                parity ^= 1;

                // 1. partial dot products of the staged rows
                // A chunk whose NR rows are all live takes loops without predicates, which the compiler is free to
                // interleave: a lane whose slice lies past the row's end reads whatever the buffer holds there
                // (finite once widened) against a centre value of zero.
                const bool full = live == (NR == 32 ? 0xFFFFFFFFu : (1u << NR) - 1u);
                double xp[CR];
#pragma unroll
                for (int j = 0; j < CR; ++j) xp[j] = 0.0;   // rows NR .. CR-1 of a whole chunk stay zero
                if (full) {
#pragma unroll
                    for (int i = 0; i < NV; ++i) {
                        float f[NR][VW];
#pragma unroll
                        for (int j = 0; j < NR; ++j) Slice<VW>::load(stage + (size_t)j * stride + (lane + 32 * i) * VW, f[j]);
#pragma unroll
                        for (int c = 0; c < VW; ++c)
#pragma unroll
                            for (int j = 0; j < NR; ++j) xp[j] = fma(widen_down(f[j][c]), v[i][c], xp[j]);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < CR; ++j) {
                        if ((live >> j) & 1u) {
                            const float* __restrict__ u = stage + (size_t)j * stride;
#pragma unroll
                            for (int i = 0; i < NV; ++i) {
                                const uint32_t e = lane + 32 * i;
                                if (e < dv) {
                                    float f[VW];
                                    Slice<VW>::load(u + e * VW, f);
#pragma unroll
                                    for (int c = 0; c < VW; ++c) xp[j] = fma(widen_down(f[c]), v[i][c], xp[j]);
                                }
                            }
                        }
                    }
                }
                // 2. transposing reduction: after it the 32 / CR lanes [j * LPR, (j + 1) * LPR) hold the dot product of row j
                constexpr int LPR = 32 / CR;
#pragma unroll
                for (int h = CR / 2, off = 16; h >= 1; h >>= 1, off >>= 1) {
                    const bool up = lane & off;
#pragma unroll
                    for (int i = 0; i < h; ++i) {
                        const double keep = up ? xp[h + i] : xp[i], give = up ? xp[i] : xp[h + i];
                        xp[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, give, off);
                    }
                }
                double x = xp[0];
#pragma unroll
                for (int off = LPR / 2; off >= 1; off >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, off);
                // 3. gradient scalar and loss of row (lane / LPR), all rows at once
                const uint32_t jr = lane / LPR;
                const bool writer = (lane % LPR) == 0;
                double g = 0.0;
                if ((live >> jr) & 1u) {
                    const bool positive = j0 + jr == 0;
                    const SigmoidLoss sl = sigmoid_loss(x);
                    g = positive ? sl.sig - 1.0 : sl.sig;
                    const double y = positive ? x : -x;   // the term is -log(sigmoid(y))
                    if (writer) loss += (y < 0.0 ? -y : 0.0) + sl.softplus;
                }
                if (writer && jr < nr && in_bounds(lim, (uint64_t)cbase + j0 + jr, lim.contrib)) rec[cbase + j0 + jr] = Rec{g, centre, 0u};
                // 4. centre gradient: acc += g_j * u_j
                if (full) {
                    double gw[NR];
#pragma unroll
                    for (int j = 0; j < NR; ++j) gw[j] = __shfl_sync(0xFFFFFFFFu, g, LPR * j) * kWidenUp;   // exact: |g| <= 1
#pragma unroll
                    for (int i = 0; i < NV; ++i) {
#pragma unroll
                        for (int j = 0; j < NR; ++j) {
                            float f[VW];
                            Slice<VW>::load(stage + (size_t)j * stride + (lane + 32 * i) * VW, f);
#pragma unroll
                            for (int c = 0; c < VW; ++c) acc[i][c] = fma(gw[j], widen_down(f[c]), acc[i][c]);
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < CR; ++j) {
                        const double gj = __shfl_sync(0xFFFFFFFFu, g, LPR * j) * kWidenUp;
                        if ((live >> j) & 1u) {
                            const float* __restrict__ u = stage + (size_t)j * stride;
#pragma unroll
                            for (int i = 0; i < NV; ++i) {
                                const uint32_t e = lane + 32 * i;
                                if (e < dv) {
                                    float f[VW];
                                    Slice<VW>::load(u + e * VW, f);
#pragma unroll
                                    for (int c = 0; c < VW; ++c) acc[i][c] = fma(gj, widen_down(f[c]), acc[i][c]);
                                }
                            }
                        }
                    }
                }
            }
        }
        if (failed || !in_bounds(lim, 2ull * q + side, lim.positions)) break;
        double2* out = reinterpret_cast<double2*>(gin_pos + (size_t)(2 * q + side) * stride);
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const uint32_t e = lane + 32 * i;
            if (e < dv) {
#pragma unroll
                for (int c = 0; c < VW; c += 2) out[(e * VW + c) / 2] = make_double2(acc[i][c], acc[i][c + 1]);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xFFFFFFFFu, loss, o);
        if (lane == 0) loss_pos[2 * q + side] = loss;
    }
    if (failed && lane == 0) atomicOr(err, kErrTimeout);
}

// Launch shape of the forward kernel: rows reduced together (8 by default: less shared memory per warp, so
// more resident warps; or 16) and blocks per multiprocessor; both can be overridden for sweeps.
static int g_forward_rows = 0;     // 0 = choose
static int g_forward_blocks = 0;   // 0 = choose
void set_forward_shape(int rows, int blocks_per_sm) {
    g_forward_rows = rows;
    g_forward_blocks = blocks_per_sm;
}

cudaError_t launch_forward(const Launcher& L, const int32_t* tok, uint32_t n, const Shape& s, const float* table,
                           const uint32_t* rows, Rec* rec, double* gin_pos, double* loss_pos, uint32_t* err,
                           const uint32_t* owned, const uint32_t* n_owned, const uint32_t* batch_err, bool sort_runs_beside) {
    if (n < 2) return cudaSuccess;
    if (L.device < 0 || L.device >= kMaxDevices) return cudaErrorInvalidDevice;
    const size_t row = (size_t)s.stride * 4;
    const int cr = g_forward_rows == 4 || g_forward_rows == 8 || g_forward_rows == 16 ? g_forward_rows : 8;
    int blocks_per_sm = g_forward_blocks > 0 ? g_forward_blocks : (cr == 16 ? 5 : cr == 8 ? 8 : 10);
    // rows staged per chunk: as many of the cr as fit the shared memory share of one block
    uint32_t chunk_rows = s.K1 < (uint32_t)cr ? s.K1 : (uint32_t)cr;
    // Slices of 2 floats where they leave fewer lanes idle than slices of 4 (an odd number of rounds of 64 floats,
    // up to 7 of them); nv = rounds of 32 lanes.
    const uint32_t rounds2 = (s.d / 2 + 31) / 32, rounds4 = (s.d4 + 31) / 32;
    const int vw = rounds2 * 2 < rounds4 * 4 && rounds2 <= 7 ? 2 : 4;
    const uint32_t nv = vw == 2 ? rounds2 : (rounds4 <= 4 ? rounds4 : 8);
    // a warp's buffer ends with padding up to slice 32 * nv of its last row (see the kernel)
    const size_t pad = 32u * nv * vw * 4 > row ? 32u * nv * vw * 4 - row : 0;
    // Whole chunks first: the loops without predicates need all cr rows staged, and they are worth more than
    // resident blocks (measured at d = 512: 6 blocks of whole chunks 0.89 ms, 8 blocks of 6-row chunks 1.15 ms).
    auto fits = [&](uint32_t rows_, int blocks_) {
        return (size_t)kFwdWarps * (rows_ * row + pad) + kFwdWarps * 8 <= (size_t)216 * 1024 / blocks_ - 1024;
    };
    if (g_forward_blocks <= 0)
        while (blocks_per_sm > 2 && !fits(chunk_rows, blocks_per_sm)) --blocks_per_sm;
    const size_t budget = (size_t)216 * 1024 / blocks_per_sm - 1024;
    while (chunk_rows > 1 && (size_t)kFwdWarps * (chunk_rows * row + pad) + kFwdWarps * 8 > budget) --chunk_rows;
    const uint32_t warp_stage = (uint32_t)((chunk_rows * row + pad) / 4);
    const size_t smem = (size_t)kFwdWarps * warp_stage * 4 + kFwdWarps * 8;
    if (smem > 200 * 1024) return cudaErrorInvalidConfiguration;
    uint32_t blocks = (2 * n + kFwdWarps - 1) / kFwdWarps;
    const uint32_t resident = (uint32_t)(L.sms * blocks_per_sm);
    if (blocks > resident) blocks = resident;
    Timed timed(L, K_FORWARD);
#define TENSAIR_FWD(NV, CR, NR, VW)                                                                                 \
    do {                                                                                                            \
        /* function attributes belong to a device: set them once on each device that launches */                  \
        static bool attr_set_on[kMaxDevices] = {};                                                                  \
        static int room_for_on[kMaxDevices] = {};                                                                   \
        bool& attr_set = attr_set_on[L.device];                                                                     \
        int& room_for = room_for_on[L.device];                                                                      \
        if (!attr_set) {                                                                                            \
            cudaFuncSetAttribute(k_forward<NV, CR, NR, VW>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024); \
            cudaFuncSetAttribute(k_forward<NV, CR, NR, VW>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);   \
            cudaFuncAttributes fa;                                                                                  \
            if (cudaFuncGetAttributes(&fa, k_forward<NV, CR, NR, VW>) == cudaSuccess && fa.numRegs > 0)             \
                room_for = (65536 - kRegistersLeftForTheSort) / (fa.numRegs * kFwdWarps * 32);                      \
            attr_set = true;                                                                                        \
        }                                                                                                           \
        uint32_t grid = blocks;                                                                                     \
        if (g_forward_blocks <= 0 && grid_shape().overlap_sort && sort_runs_beside && room_for >= 1 &&              \
            grid > (uint32_t)(L.sms * room_for))                                                                    \
            grid = (uint32_t)(L.sms * room_for);                                                                    \
        k_forward<NV, CR, NR, VW><<<grid, kFwdWarps * 32, smem, L.stream>>>(tok, n, s.V, s.d, s.stride, s.w, s.k,   \
                                                                            chunk_rows, warp_stage, table, rows,    \
                                                                            rec, gin_pos, loss_pos, err, owned,     \
                                                                            n_owned, batch_err, L.lim);             \
    } while (0)
    // k = 5 (six rows per pair) is common enough to have whole chunks of its own
#define TENSAIR_FWD_ROWS(NV, VW)                                                     \
    do {                                                                             \
        if (cr == 16) TENSAIR_FWD(NV, 16, 16, VW);                                   \
        else if (cr == 8 && chunk_rows == 6) TENSAIR_FWD(NV, 8, 6, VW);              \
        else if (cr == 8) TENSAIR_FWD(NV, 8, 8, VW);                                 \
        else TENSAIR_FWD(NV, 4, 4, VW);                                              \
    } while (0)
    if (vw == 2) {
        if (nv == 1) TENSAIR_FWD_ROWS(1, 2);
        else if (nv == 3) TENSAIR_FWD_ROWS(3, 2);
        else if (nv == 5) TENSAIR_FWD_ROWS(5, 2);
        else TENSAIR_FWD_ROWS(7, 2);
    } else {
        if (nv == 1) TENSAIR_FWD_ROWS(1, 4);
        else if (nv == 2) TENSAIR_FWD_ROWS(2, 4);
        else if (nv == 3) TENSAIR_FWD_ROWS(3, 4);
        else if (nv == 4) TENSAIR_FWD_ROWS(4, 4);
        else TENSAIR_FWD_ROWS(8, 4);
    }
#undef TENSAIR_FWD_ROWS
#undef TENSAIR_FWD
    return cudaGetLastError();
}

// Sum of the losses of the 2n half positions (in a routed batch: of the replica's own positions) in a fixed order, in fp64.
__global__ void __launch_bounds__(1024)
k_loss_sum(const double* __restrict__ loss_pos, uint32_t n, double* __restrict__ loss, const uint32_t* __restrict__ err,
           const uint8_t* __restrict__ owner) {
    __shared__ double part[1024];
    double s = 0.0;
    if (!*err)
        for (uint32_t i = threadIdx.x; i < 2 * n; i += 1024)
            if (!owner || owner[i >> 1]) s += loss_pos[i];
    part[threadIdx.x] = s;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss = part[0];
}

cudaError_t launch_loss_sum(const Launcher& L, const double* loss_pos, uint32_t n, double* loss, const uint32_t* err,
                            const uint8_t* owner) {
    Timed timed(L, K_LOSS_SUM);
    k_loss_sum<<<1, 1024, 0, L.stream>>>(loss_pos, n < 2 ? 0 : n, loss, err, owner);
    return cudaGetLastError();
}

}  // namespace tensair
