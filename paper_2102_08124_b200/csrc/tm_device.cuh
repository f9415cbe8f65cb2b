// Shared device-side definitions of the transposable N:M mask search kernels.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace tmask {

constexpr int kMethodExact = 0;
constexpr int kMethodApprox = 1;
constexpr int kMethodCover = 2;
constexpr int kMethodRows = 3;       // internal: plain N:M along rows (no column constraint), M = 4
constexpr int kMethodRowsAbsorb = 4; // internal: the same with the mean of the pruned weights absorbed into the kept ones
constexpr int kF32 = 0;
constexpr int kBF16 = 1;
constexpr int kDevNonFinite = 1;
constexpr int kDevInternal = 2;
constexpr int kDevBadMask = 4;

// One matrix of a (possibly batched) call, as the kernels see it.
struct DevProblem {
    const void* W;
    uint32_t* mask;
    void* masked;        // may be null, may alias W
    double* objective;   // may be null
    long long rows, cols, ld;
    long long item_begin;  // index of this problem's first work item in the call-wide numbering
    int dtype;
    int wpr;             // mask words per row
    int bcols;           // blocks per block row
    int chunks;          // work items per block row
};

// One matrix of the neighbouring operations (1-D pruning, violation count, 2:4 compression).
struct AuxProblem {
    const void* W;
    uint32_t* mask;      // output of the 1-D pruning, input of the other two
    void* masked;        // may be null
    long long rows, cols, ld;
    int dtype;
    int wpr;
};

// Magnitudes travel as the fp32 bit pattern of |w| (bf16 widened exactly): for finite values the
// unsigned order of the patterns is the order of |w|, and -0 == +0.
__device__ __forceinline__ float pattern_as_float(uint32_t u) { return __uint_as_float(u); }

__device__ __forceinline__ float bf16_to_float(uint32_t h) { return __uint_as_float(h << 16); }
// fp32 -> bf16, round to nearest even; NaN stays NaN
__device__ __forceinline__ uint32_t float_to_bf16_bits(float f) {
    const uint32_t u = __float_as_uint(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (u >> 16) | 0x40u;
    return (u + 0x7FFFu + ((u >> 16) & 1u)) >> 16;
}

}  // namespace tmask
