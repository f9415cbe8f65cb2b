// Host-side launch interface between the C ABI (tm_api.cu) and the kernel translation units.
#pragma once
#include "tm_device.cuh"

namespace tmask {

struct LaunchArgs {
    DevProblem single;          // used when table == nullptr (count == 1)
    const DevProblem* table;    // device array of `count` problems, or nullptr
    int count;
    long long total_items;
    double* partials;           // device scratch, count * ctas * warps-per-CTA doubles
    int* status;                // device int or nullptr
    int ctas;
    int N, M, method;
    cudaStream_t stream;
};

// Generic path: any supported (N, M, method, dtype, ld).  Zeroes the partials, runs the search and
// the fixed-order objective reduction on a.stream.
cudaError_t launch_generic(const LaunchArgs& a);
int generic_warps_per_cta();

}  // namespace tmask
