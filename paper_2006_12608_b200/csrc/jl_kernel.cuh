// The random-sign level matrices of the JL transform (Section 3): M = (I_{r_l} (x) A_l) ... (I_{r_1} (x) A_1).
// A_i is k_i x c_i with independent +-1 entries (scaled by 1/sqrt(k_i) where the product is stored); the sign
// of entry (a, b) is bit 0 of splitmix64(seed, i * 2^40 + a * c_i + b) -- counter-based, nothing is stored
// between calls.  Applying a level is a dense product handled by the tile kernel (KIND_STORE).
#pragma once
#include <cstdint>

#include "lsh_kernel.cuh"   // lsh_splitmix64

namespace sj {

// A (k_i x c_i, row-major bf16): +1.0 = 0x3f80, -1.0 = 0xbf80.
__global__ void __launch_bounds__(256) jl_sign_matrix_kernel(unsigned long long seed, int level, int k_i, int c_i,
                                                             uint16_t *__restrict__ A) {
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (long long)k_i * c_i) return;
    const uint64_t bits = lsh_splitmix64(seed, ((uint64_t)level << 40) + (uint64_t)t);
    A[t] = (bits & 1u) ? 0x3f80u : 0xbf80u;
}

}  // namespace sj
