// Hashing shared by the selection kernels: the shared random-k index set
// (Sec. 5.3: same seed on every GPU) and the count sketch's h_i, s_i
// (Sec. 4.2.2) come from one 64-bit finalising mixer (splitmix64's) keyed by
// (seed, a, b) and evaluated at the element index.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace conef {

__host__ __device__ __forceinline__ uint64_t mix64(uint64_t z)
{
    z ^= z >> 30;
    z *= 0xBF58476D1CE4E5B9ULL;
    z ^= z >> 27;
    z *= 0x94D049BB133111EBULL;
    z ^= z >> 31;
    return z;
}
constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ULL;
__host__ __device__ __forceinline__ uint64_t stream_key(uint64_t seed, uint64_t a, uint64_t b)
{
    return mix64(mix64(seed + kGolden * (a + 1)) + kGolden * (b + 1));
}
__host__ __device__ __forceinline__ uint64_t h64(uint64_t st, uint64_t j)
{
    return mix64(st + kGolden * (j + 1));
}
__device__ __forceinline__ uint32_t hash32(uint64_t st, uint64_t j) { return (uint32_t)(h64(st, j) >> 32); }


// membership in S_t: key(j) = (hash32(j) << 32) | j is not above the threshold (tau_hi, tau_lo)
__device__ __forceinline__ bool rk_selected(uint32_t h, uint32_t j, uint32_t tau_hi, uint32_t tau_lo)
{
    return h < tau_hi || (h == tau_hi && j <= tau_lo);
}

// random-block-k: first index of the kept block, uniform on [0, d - k], from the shared stream
__host__ __device__ __forceinline__ uint32_t randblock_start(uint64_t st, uint32_t d, uint32_t k)
{
    return (uint32_t)(((h64(st, 0) >> 32) * ((uint64_t)(d - k) + 1)) >> 32);
}

}  // namespace conef
