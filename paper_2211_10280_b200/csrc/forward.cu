// Gradient calculation at the snapshot: fused gather -> dot -> sigmoid -> gradient scalars, centre-stationary.
// Rows are fp32 in memory; the dot products, the sigmoid and the partial sums are taken in fp64.
//
// One block per centre position q.  Each warp takes window slots of that position; for a slot it keeps
// the centre row v_c in registers, gathers the 1 + k output rows of the pair (positive first), reduces
// each dot product with warp shuffles, turns it into the gradient scalar g (sigma(x) - 1 for the
// positive, sigma(x) for a negative, 0 for a negative equal to the positive), records g for the later
// per-output-row sums and accumulates g * u into the centre's own gradient while the row is still in
// registers - the output rows are read from memory exactly once per contribution.  The block then adds
// its warps' partial sums in warp order and writes one partial centre gradient per position.
#include "kernels.h"

namespace tensair {


// -log(sigmoid(-z)) = log(1 + e^z), without overflow
__device__ inline double softplus(double z) { return fmax(z, 0.0) + log1p(exp(-fabs(z))); }

// NV: float4 slices per lane; RIF: output rows a warp loads before it starts reducing.
template <int NV, int RIF>
__global__ void __launch_bounds__(384)
k_forward(const int32_t* __restrict__ tok, uint32_t n, uint32_t V, uint32_t d4, uint32_t stride4, uint32_t w,
          uint32_t k, const float4* __restrict__ table, const uint32_t* __restrict__ rows, Rec* __restrict__ rec,
          double* __restrict__ gin_pos, double* __restrict__ loss_pos, const uint32_t* __restrict__ err) {
    if (*err) return;
    extern __shared__ double smem[];          // [warps][4*d4] partial centre gradients, then [warps] losses
    const uint32_t lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    double* loss_s = smem + (size_t)nwarps * d4 * 4;
    const uint32_t q = blockIdx.x;
    const uint32_t centre = (uint32_t)tok[q];
    const uint32_t K1 = k + 1;
    const float4* __restrict__ vin = table + (size_t)centre * stride4;
    const float4* __restrict__ tout = table + (size_t)V * stride4;

    // the centre row and this warp's partial gradient, both in fp64
    double v[NV][4], acc[NV][4];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const uint32_t e = lane + 32 * i;
        const float4 f = e < d4 ? __ldg(vin + e) : make_float4(0.f, 0.f, 0.f, 0.f);
        v[i][0] = (double)f.x; v[i][1] = (double)f.y; v[i][2] = (double)f.z; v[i][3] = (double)f.w;
        acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.0;
    }
    double loss = 0.0;
    const uint32_t lo = q > w ? q - w : 0;
    const uint32_t pbase = pair_offset(q, n, w);

    for (uint32_t s = wid; s < 2 * w; s += nwarps) {
        const int64_t c = (int64_t)q + (s < w ? (int64_t)s - (int64_t)w : (int64_t)s - (int64_t)w + 1);
        if (c < 0 || c >= (int64_t)n) continue;
        const uint32_t p = pbase + ((uint32_t)c - lo) - ((uint32_t)c > q ? 1u : 0u);
        const uint32_t cbase = p * K1;
        const uint32_t ctx = (uint32_t)tok[c];
        for (uint32_t j0 = 0; j0 < K1; j0 += RIF) {
            uint32_t r[RIF];
            bool live[RIF];
            float4 u[RIF][NV];
#pragma unroll
            for (int t = 0; t < RIF; ++t) {
                const uint32_t j = j0 + t;
                r[t] = j < K1 ? __ldg(rows + cbase + j) : ctx;
                live[t] = j < K1 && (j == 0 || r[t] != ctx);
            }
#pragma unroll
            for (int t = 0; t < RIF; ++t) {
                const float4* __restrict__ urow = tout + (size_t)r[t] * stride4;
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const uint32_t e = lane + 32 * i;
                    u[t][i] = (live[t] && e < d4) ? __ldg(urow + e) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int t = 0; t < RIF; ++t) {
                const uint32_t j = j0 + t;
                if (j >= K1) break;
                double ud[NV][4];
                double x = 0.0;
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    ud[i][0] = (double)u[t][i].x; ud[i][1] = (double)u[t][i].y;
                    ud[i][2] = (double)u[t][i].z; ud[i][3] = (double)u[t][i].w;
                    x = fma(ud[i][0], v[i][0], x);
                    x = fma(ud[i][1], v[i][1], x);
                    x = fma(ud[i][2], v[i][2], x);
                    x = fma(ud[i][3], v[i][3], x);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xFFFFFFFFu, x, o);
                double g = 0.0;
                if (live[t]) {
                    const double sig = 1.0 / (1.0 + exp(-x));
                    g = j == 0 ? sig - 1.0 : sig;
                    loss += softplus(j == 0 ? -x : x);
#pragma unroll
                    for (int i = 0; i < NV; ++i) {
                        acc[i][0] = fma(g, ud[i][0], acc[i][0]);
                        acc[i][1] = fma(g, ud[i][1], acc[i][1]);
                        acc[i][2] = fma(g, ud[i][2], acc[i][2]);
                        acc[i][3] = fma(g, ud[i][3], acc[i][3]);
                    }
                }
                if (lane == 0) rec[cbase + j] = Rec{g, centre, 0u};
            }
        }
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const uint32_t e = lane + 32 * i;
        if (e < d4) {
            double* dst = smem + ((size_t)wid * d4 + e) * 4;
            dst[0] = acc[i][0]; dst[1] = acc[i][1]; dst[2] = acc[i][2]; dst[3] = acc[i][3];
        }
    }
    if (lane == 0) loss_s[wid] = loss;
    __syncthreads();
    const uint32_t dd = d4 * 4;
    for (uint32_t e = threadIdx.x; e < dd; e += blockDim.x) {
        double sum = smem[e];
        for (uint32_t x = 1; x < nwarps; ++x) sum += smem[(size_t)x * dd + e];
        gin_pos[(size_t)q * stride4 * 4 + e] = sum;
    }
    if (threadIdx.x == 0) {
        double l = loss_s[0];
        for (uint32_t x = 1; x < nwarps; ++x) l += loss_s[x];
        loss_pos[q] = l;
    }
}

cudaError_t launch_forward(const Launcher& L, const int32_t* tok, uint32_t n, const Shape& s, const float* table,
                           const uint32_t* rows, Rec* rec, double* gin_pos, double* loss_pos, const uint32_t* err) {
    if (n < 2) return cudaSuccess;
    uint32_t warps = 2 * s.w;
    if (warps > 12) warps = 12;
    const uint32_t fit = 49152 / (s.d * 8 + 8);   // partial sums and losses within 48 KB of shared memory
    if (warps > fit) warps = fit;
    if (warps < 1) warps = 1;
    const size_t smem = ((size_t)warps * s.d + warps) * sizeof(double);
    const uint32_t stride4 = s.stride / 4;
    const float4* t4 = reinterpret_cast<const float4*>(table);
    Timed timed(L, K_FORWARD);
#define TENSAIR_FWD(NV, RIF) \
    k_forward<NV, RIF><<<n, warps * 32, smem, L.stream>>>(tok, n, s.V, s.d4, stride4, s.w, s.k, t4, rows, rec, gin_pos, loss_pos, err)
    if (s.d4 <= 32) TENSAIR_FWD(1, 4);
    else if (s.d4 <= 64) TENSAIR_FWD(2, 4);
    else if (s.d4 <= 96) TENSAIR_FWD(3, 4);
    else if (s.d4 <= 128) TENSAIR_FWD(4, 2);
    else TENSAIR_FWD(8, 1);
#undef TENSAIR_FWD
    return cudaGetLastError();
}

// Sum of the per-position losses in a fixed order, in fp64.
__global__ void __launch_bounds__(1024)
k_loss_sum(const double* __restrict__ loss_pos, uint32_t n, double* __restrict__ loss, const uint32_t* __restrict__ err) {
    __shared__ double part[1024];
    double s = 0.0;
    if (!*err)
        for (uint32_t i = threadIdx.x; i < n; i += 1024) s += loss_pos[i];
    part[threadIdx.x] = s;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if ((int)threadIdx.x < o) part[threadIdx.x] += part[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *loss = part[0];
}

cudaError_t launch_loss_sum(const Launcher& L, const double* loss_pos, uint32_t n, double* loss, const uint32_t* err) {
    Timed timed(L, K_LOSS_SUM);
    k_loss_sum<<<1, 1024, 0, L.stream>>>(loss_pos, n < 2 ? 0 : n, loss, err);
    return cudaGetLastError();
}

}  // namespace tensair
