// Work-item bookkeeping shared by the bandwidth kernels: one descriptor record per matrix (tensor maps
// for loads and stores plus the problem), a cursor that walks the items of a table of matrices in
// order, and the host-side construction of the records.  An item is one block row of the matrix wide enough
// to fill a stage: 4 rows x 512 columns for M = 4, 8 rows x 256 columns for M = 8.
#pragma once
#include <cstring>

#include "tm_device.cuh"
#include "tm_tma.cuh"

namespace tmask {

struct alignas(128) TmaEntry {
    CUtensorMap in, out;
    DevProblem p;
    int cchunks;       // items per item row
    int brows;         // item rows (one block row of the matrix each)
};
static_assert(sizeof(TmaEntry) == 384 || sizeof(TmaEntry) == 512, "descriptor records stay 128-byte aligned in tables");

// Even split of `total` work items over the warps of the grid: every warp gets total / nwarps items and the first
// total % nwarps warps one more -- "first" in an order that runs across the CTAs before it runs down their warps, so
// that the surplus items fall on as many different SMs as possible (an SM's warps share its issue slots: what counts
// is the SM's total).  Returns the warp's first item and sets its item count.
__device__ __forceinline__ long long even_share(long long total, int warps_per_cta, int& n_items) {
    const long long nwarps = (long long)gridDim.x * warps_per_cta;
    const long long order = (long long)(threadIdx.x >> 5) * gridDim.x + blockIdx.x;
    const long long q = total / nwarps, rem = total - q * nwarps;
    n_items = (int)(q + (order < rem ? 1 : 0));
    return order * q + (order < rem ? order : rem);
}

// The matrix that holds work item `item`: the last record whose first item is not beyond it (first items never
// decrease along the table).  Called by all 32 lanes of a warp with the same arguments: every lane tests its own
// records, so a table of a hundred matrices costs three independent loads per lane instead of a hundred dependent ones.
__device__ __forceinline__ int find_matrix(const TmaEntry* tab, int count, long long item) {
    const int lane = threadIdx.x & 31;
    int n = 0;
    for (int base = 1; base < count; base += 32) {
        const int k = base + lane;
        const bool reached = k < count && tab[k].p.item_begin <= item;
        n += __popc(__ballot_sync(0xFFFFFFFFu, reached));
    }
    return n;
}

// End of a single-matrix launch that reduces its own objective (`done` is a 32-bit count in device memory that is zero when
// the launch starts).  Every warp of the grid has stored its partial sum -- a zero if it had no work item -- at
// partials[its index]; all threads of the CTA call this once, as the last thing they do.  The CTA that arrives last adds the
// nwarps partials in an order that depends on nothing but nwarps and the CTA's size (so the same launch gives the same
// bits whichever CTA that is), writes the objective and sets the count back to zero for the next launch.  Nobody waits for
// anybody: the earlier CTAs just leave.  `scratch`: 33 doubles of shared memory that nothing else uses any more.
#ifndef TMX_FIN
#define TMX_FIN static __device__ __noinline__
#endif
TMX_FIN void finish_objective(unsigned int* done, const double* partials, long long nwarps, double* objective, double* scratch) {
    volatile int* is_last = reinterpret_cast<volatile int*>(scratch + 32);
    __threadfence();                                   // my warp's partial is visible to the grid before the CTA is counted
    __syncthreads();
    if (threadIdx.x == 0) *is_last = atomicAdd(done, 1u) == gridDim.x - 1 ? 1 : 0;
    __syncthreads();
    if (!*is_last) return;
    __threadfence();
    double s = 0.0;
    for (long long i = threadIdx.x; i < nwarps; i += blockDim.x) s += __ldcg(partials + i);
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += scratch[w];
        if (objective) *objective = t;
        *done = 0u;
    }
}

// The same for a launch over several matrices whose warps hold contiguous item ranges dealt by even_share().  A warp that
// worked on matrix k has stored its partial sum for it at partials[order + k] (order = its place in even_share()'s order;
// the pairs (order, k) of a launch are strictly increasing in both, so the slots are distinct and number at most
// nwarps + count), and nothing else is ever read: which warps worked on matrix k follows from its first and last item, so
// the buffer needs no clearing.  The CTA that arrives last gives every matrix to one of its warps, which adds the matrix's
// partials in a fixed order.
__device__ __forceinline__ long long even_share_owner(long long item, long long q, long long rem) {
    return item < rem * (q + 1) ? item / (q + 1) : rem + (item - rem * (q + 1)) / q;
}
TMX_FIN void finish_objectives_ranged(unsigned int* done, const double* partials, const TmaEntry* tab, int count,
                                      long long total_items, long long nwarps, double* scratch) {
    volatile int* is_last = reinterpret_cast<volatile int*>(scratch);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *is_last = atomicAdd(done, 1u) == gridDim.x - 1 ? 1 : 0;
    __syncthreads();
    if (!*is_last) return;
    __threadfence();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    const long long q = total_items / nwarps, rem = total_items - q * nwarps;
    for (int k = warp; k < count; k += warps) {
        const long long n = (long long)tab[k].brows * tab[k].cchunks, begin = tab[k].p.item_begin;
        double s = 0.0;
        if (n > 0) {
            const long long o0 = even_share_owner(begin, q, rem), o1 = even_share_owner(begin + n - 1, q, rem);
            for (long long o = o0 + lane; o <= o1; o += 32) s += __ldcg(partials + o + k);
        }
        for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
        if (lane == 0 && tab[k].p.objective) *tab[k].p.objective = s;
    }
    __syncthreads();
    if (threadIdx.x == 0) *done = 0u;
}

// Walks the work items of a table of problems in order: problem k, block row bi, column chunk cj.
struct Cursor {
    int k, bi, cj, cchunks, brows;
    __device__ __forceinline__ void load(const TmaEntry* tab, int count) {
        while (k < count && (tab[k].brows == 0 || tab[k].cchunks == 0)) ++k;   // empty matrices have no items
        if (k < count) { cchunks = tab[k].cchunks; brows = tab[k].brows; } else { cchunks = 1; brows = 1; }
    }
    __device__ __forceinline__ void seek(const TmaEntry* tab, int count, long long item) {
        k = find_matrix(tab, count, item);
        load(tab, count);
        const long long local = item - tab[k < count ? k : count - 1].p.item_begin;
        bi = (int)(local / cchunks); cj = (int)(local - (long long)bi * cchunks);
    }
    __device__ __forceinline__ void advance(const TmaEntry* tab, int count) {
        if (++cj == cchunks) {
            cj = 0;
            if (++bi == brows) { bi = 0; ++k; load(tab, count); }
        }
    }
};

// The same walk in steps of `stride` items (the warps of a launch take the items round-robin, so that at any
// moment the whole grid works on one dense window of the matrix).  Inside a matrix a step is an addition;
// only the step that leaves a matrix goes through the item index.
struct StrideCursor {
    int k, bi, cj, cchunks, brows, dbi, dcj, stride;
    __device__ __forceinline__ void enter(const TmaEntry* tab, int count) {
        while (k < count && (tab[k].brows == 0 || tab[k].cchunks == 0)) ++k;   // empty matrices have no items
        if (k < count) { cchunks = tab[k].cchunks; brows = tab[k].brows; } else { cchunks = 1; brows = 1; }
        dbi = stride / cchunks; dcj = stride - dbi * cchunks;
    }
    __device__ __forceinline__ void seek(const TmaEntry* tab, int count, long long item, int stride_) {
        stride = stride_;
        k = find_matrix(tab, count, item);
        enter(tab, count);
        const long long local = item - tab[k < count ? k : count - 1].p.item_begin;
        bi = (int)(local / cchunks); cj = (int)(local - (long long)bi * cchunks);
    }
    __device__ __forceinline__ void advance(const TmaEntry* tab, int count) {
        cj += dcj; bi += dbi;
        if (cj >= cchunks) { cj -= cchunks; ++bi; }
        if (bi >= brows) {
            long long over = (long long)(bi - brows) * cchunks + cj;             // items past the end of matrix k
            for (;;) {
                ++k; enter(tab, count);
                if (k >= count) { bi = 0; cj = 0; break; }
                const long long n = (long long)brows * cchunks;
                if (over < n) { bi = (int)(over / cchunks); cj = (int)(over - (long long)bi * cchunks); break; }
                over -= n;
            }
        }
    }
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) { cudaGetLastError(); p = nullptr; }
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// A box is at most 256 elements wide, so a wider item is described in units of 2 or 4 matrix elements (the
// copy moves bytes; rows are 16-byte multiples and the column count a multiple of M, so the units divide
// evenly and the zero fill past the last column falls on whole units).  The x coordinate of item cj is
// cj * kTmaBoxUnits for every item shape.
constexpr int kTmaBoxUnits = 256;
inline bool encode_map(CUtensorMap* m, const void* base, int dtype, long long rows, long long cols, long long ld, int box_rows, int box_cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const int esz = dtype == kF32 ? 4 : 2;
    const int unit = box_cols * esz / kTmaBoxUnits;                      // bytes per tensor-map element: 2, 4 or 8
    if (unit != 2 && unit != 4 && unit != 8) return false;
    if ((cols * esz) % unit) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)(cols * esz / unit), (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * esz};
    const cuuint32_t box[2] = {(cuuint32_t)kTmaBoxUnits, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType type = unit == 2 ? CU_TENSOR_MAP_DATA_TYPE_UINT16 : (unit == 4 ? CU_TENSOR_MAP_DATA_TYPE_UINT32 : CU_TENSOR_MAP_DATA_TYPE_UINT64);
    return fn(m, type, 2, const_cast<void*>(base), dims, strides,
              box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


inline bool build_entries(const DevProblem* probs, int count, TmaEntry* e, long long* total_items, int item_rows, int item_cols) {
    long long total = 0;
    for (int k = 0; k < count; ++k) {
        memset(&e[k], 0, sizeof(TmaEntry));
        e[k].p = probs[k];
        e[k].cchunks = (int)((probs[k].cols + item_cols - 1) / item_cols);
        e[k].brows = (int)((probs[k].rows + item_rows - 1) / item_rows);
        e[k].p.item_begin = total;
        total += (long long)e[k].brows * e[k].cchunks;
        if (probs[k].rows == 0 || probs[k].cols == 0) continue;
        if (!encode_map(&e[k].in, probs[k].W, probs[k].dtype, probs[k].rows, probs[k].cols, probs[k].ld, item_rows, item_cols)) return false;
        if (probs[k].masked) {
            if (!encode_map(&e[k].out, probs[k].masked, probs[k].dtype, probs[k].rows, probs[k].cols, probs[k].ld, item_rows, item_cols)) return false;
        } else {
            e[k].out = e[k].in;
        }
    }
    *total_items = total;
    return true;
}

}  // namespace tmask
