// Host-side launch interface between the C ABI (tm_api.cu) and the kernel translation units.
#pragma once
#include <atomic>

#include "tm_device.cuh"

namespace tmask {

// Function attributes (the dynamic shared-memory limit) belong to a device, not to the process: one flag per
// device (up to 64, the library's limit) and kernel instantiation.  Two threads that meet an unset flag both set
// the attribute, which is harmless.
struct PerDeviceOnce {
    std::atomic<unsigned long long> done{0};
    template <class Fn> cudaError_t run(Fn&& fn) {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        const unsigned long long bit = 1ull << (dev & 63);
        if (done.load(std::memory_order_acquire) & bit) return cudaSuccess;
        if ((e = fn()) != cudaSuccess) return e;
        done.fetch_or(bit, std::memory_order_release);
        return cudaSuccess;
    }
};

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
int generic_warps_per_cta(int N, int M, int method);
int generic_ctas_per_sm(int N, int M, int method);

// Bandwidth path (TMA-staged, bit-parallel): approximate 2:4 search on 16-byte aligned matrices.
struct TmaLaunch {
    const void* entries_host;   // `count` records of tma_entry_bytes() each, built by tma_build_entries()
    const void* entries_dev;    // the same records in device memory, or nullptr when count == 1
    int count;
    long long total_items;
    double* partials;           // device scratch, count * ctas * tma_warps_per_cta(dtype, M, method) doubles
    int* status;
    int ctas;
    int dtype, method, M;
    bool has_out;               // masked_w_out present (all problems of one launch agree)
    int n_keep = 2;             // kMethodRows / kMethodRowsAbsorb: entries kept per group of four (1..3)
    unsigned long long* vpartials = nullptr;   // kMethodRows / kMethodRowsAbsorb (count == 1): ctas * warps pattern-violation partials; the caller reduces
    unsigned int* done = nullptr;              // a device word that is zero between launches, or nullptr: with it a search is ONE launch where
                                               // it can be (the warps store partials, the CTA that finishes last adds them up) instead of three
    cudaStream_t stream;
};
size_t tma_entry_bytes();
int tma_warps_per_cta(int dtype, int M, int method);
bool tma_eligible(const DevProblem& p, int N, int M, int method);
bool tma_build_entries(const DevProblem* probs, int count, void* entries_host, long long* total_items, int M, int method);
cudaError_t tma_reduce(const void* entries_host, const void* entries_dev, int count, const double* partials, long long stride, cudaStream_t stream);
// 4:8 variant (tm_kernels_tma48.cu), reached through launch_tma()
int tma48_warps_per_cta(int dtype, int method);
int tma48_item_cols(int dtype, int method);
cudaError_t launch_tma48(const TmaLaunch& a);
// the same search for fp32 with a block split over two lanes (tm_kernels_tma48s.cu), reached through launch_tma48()
int tma48s_warps_per_cta();
int tma48s_item_cols();
cudaError_t launch_tma48s(const TmaLaunch& a);
cudaError_t launch_tma(const TmaLaunch& a);


// Neighbouring operations (tm_kernels_aux.cu)
int aux_partial_slots();
cudaError_t launch_aux_reduce(const double* obj_partials, const unsigned long long* viol_partials, int n, double* objective_out,
                              unsigned long long* violations_out, cudaStream_t stream);
cudaError_t launch_nm1d(const AuxProblem& P, int N, int M, int flags, bool violations_only, double* obj_partials,
                        unsigned long long* viol_partials, double* objective_out, unsigned long long* violations_out,
                        int* status, int sms, cudaStream_t stream);
cudaError_t launch_hamming(const uint32_t* a, const uint32_t* b, long long words, unsigned long long* partials, unsigned long long* out,
                           int sms, cudaStream_t stream);
// the streaming form of the compression for bf16 matrices with 16-byte aligned rows and mask rows (tm_kernels_compress.cu)
bool compress24_stream_eligible(const AuxProblem& P, const void* values, const void* meta, const void* meta_t);
cudaError_t launch_compress24_stream(const AuxProblem& P, void* values, uint32_t* meta, void* values_t, uint32_t* meta_t, int* status,
                                     int sms, cudaStream_t stream);
cudaError_t launch_compress24(const AuxProblem& P, void* values, uint32_t* meta, void* values_t, uint32_t* meta_t, int* status,
                              int sms, cudaStream_t stream);

}  // namespace tmask
