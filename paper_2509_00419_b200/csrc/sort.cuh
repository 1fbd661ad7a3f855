// Block-wide bitonic sort of 64-bit keys held in shared memory.
#pragma once
#include <stdint.h>

namespace lvlm {

// Sorts keys[0..P) ascending; P is a power of two; every thread of the block takes part.
__device__ __forceinline__ void block_bitonic_sort(uint64_t* keys, int P) {
    for (int k2 = 2; k2 <= P; k2 <<= 1) {
        for (int j = k2 >> 1; j > 0; j >>= 1) {
            for (int t = threadIdx.x; t < (P >> 1); t += blockDim.x) {
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
                const int l = i | j;
                const bool up = (i & k2) == 0;
                const uint64_t a = keys[i], b = keys[l];
                if ((a > b) == up) { keys[i] = b; keys[l] = a; }
            }
            __syncthreads();
        }
    }
}

inline int next_pow2(int x) { int p = 1; while (p < x) p <<= 1; return p; }

}  // namespace lvlm
