// Philox4x32-10 counter-based generator (Salmon et al., SC'11), host and device.
//
// Counter layouts used by the library (key = low and high word of the 64-bit seed):
//   negatives  counter = (pair index p, draw index j / 2, batch index, 1<<24 | replica);
//              output words 0,1 feed draw 2*(j/2), words 2,3 feed draw 2*(j/2)+1
//   delays     counter = (step, sender, receiver, 2<<24); word 0 is used
//   init       counter = (e/4 low, e/4 high, 0, 3<<24) for table element e = row*d + col; word e%4
#pragma once
#include <stdint.h>

namespace tensair {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kWeyl0 = 0x9E3779B9u;
constexpr uint32_t kWeyl1 = 0xBB67AE85u;

constexpr uint32_t kTagNegative = 1u << 24;
constexpr uint32_t kTagDelay = 2u << 24;
constexpr uint32_t kTagInit = 3u << 24;
constexpr uint32_t kTagRoute = 4u << 24;

struct Philox4 {
    uint32_t x, y, z, w;
};

__host__ __device__ inline uint32_t hi_product(uint32_t a, uint32_t b) {
#ifdef __CUDA_ARCH__
    return __umulhi(a, b);
#else
    return (uint32_t)(((unsigned long long)a * b) >> 32);
#endif
}

__host__ __device__ inline Philox4 philox4x32_10(Philox4 c, uint32_t key0, uint32_t key1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = hi_product(kPhiloxM0, c.x), lo0 = kPhiloxM0 * c.x;
        const uint32_t hi1 = hi_product(kPhiloxM1, c.z), lo1 = kPhiloxM1 * c.z;
        c = Philox4{hi1 ^ c.y ^ key0, lo1, hi0 ^ c.w ^ key1, lo0};
        key0 += kWeyl0;
        key1 += kWeyl1;
    }
    return c;
}

}  // namespace tensair
