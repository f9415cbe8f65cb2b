// Bandwidth kernels of the approximate 2:4 search (TM_APPROX / TM_APPROX_COVER, M = 4).
//
// Every warp runs its own software pipeline over a contiguous range of work items (4 rows x 256
// columns of one matrix): lane 0 keeps bulk-tensor (TMA) loads of the next items in flight into a
// private ring of shared-memory stages, the 32 lanes read their two 4x4 blocks from the landed stage
// with 128-bit shared loads, run the bit-parallel search (tm_core24.cuh) in registers, write the
// masked weights back into the same stage and lane 0 sends it out with a TMA store.  Mask bytes
// meet in shared memory and leave as whole 32-bit words.  No CTA-wide synchronisation exists; all
// waits are bounded.
#include "tm_core24.cuh"
#include "tm_launch.h"
#include "tm_tma.cuh"

#include <cstring>

namespace tmask {

namespace {

constexpr int kWarps = 16;                 // warps per CTA, one CTA per SM
constexpr int kItemRows = 4;
constexpr int kItemCols = 256;

template <int DT> struct Geometry {
    static constexpr int kElem = DT == kF32 ? 4 : 2;
    static constexpr int kStages = DT == kF32 ? 3 : 4;
    static constexpr int kStageBytes = kItemRows * kItemCols * kElem;
    static constexpr int kWarpBytes = kStages * kStageBytes + 128 /* mask bytes */ + 64 /* barriers */ + 64;
};

// 16 magnitudes of each of the lane's two blocks, as integers ordered like |w|
template <int DT>
__device__ __forceinline__ void load_keys(const unsigned char* stage, int lane, uint32_t (&raw)[4][DT == kF32 ? 8 : 4],
                                          uint32_t (&ka)[16], uint32_t (&kb)[16]) {
    if constexpr (DT == kBF16) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 v = *reinterpret_cast<const uint4*>(stage + i * (kItemCols * 2) + lane * 16);
            raw[i][0] = v.x; raw[i][1] = v.y; raw[i][2] = v.z; raw[i][3] = v.w;
            ka[4 * i + 0] = v.x & 0x7FFFu; ka[4 * i + 1] = (v.x >> 16) & 0x7FFFu; ka[4 * i + 2] = v.y & 0x7FFFu; ka[4 * i + 3] = (v.y >> 16) & 0x7FFFu;
            kb[4 * i + 0] = v.z & 0x7FFFu; kb[4 * i + 1] = (v.z >> 16) & 0x7FFFu; kb[4 * i + 2] = v.w & 0x7FFFu; kb[4 * i + 3] = (v.w >> 16) & 0x7FFFu;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 a = *reinterpret_cast<const uint4*>(stage + i * (kItemCols * 4) + lane * 32);
            const uint4 b = *reinterpret_cast<const uint4*>(stage + i * (kItemCols * 4) + lane * 32 + 16);
            raw[i][0] = a.x; raw[i][1] = a.y; raw[i][2] = a.z; raw[i][3] = a.w; raw[i][4] = b.x; raw[i][5] = b.y; raw[i][6] = b.z; raw[i][7] = b.w;
#pragma unroll
            for (int j = 0; j < 4; ++j) { ka[4 * i + j] = raw[i][j] & 0x7FFFFFFFu; kb[4 * i + j] = raw[i][4 + j] & 0x7FFFFFFFu; }
        }
    }
}

// independent halves of the relation masks from scalar keys (one block into one half of the pair masks)
__device__ __forceinline__ void relations_scalar(const uint32_t (&k)[16], int shift, Rel24& r) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t a = k[4 * i], b = k[4 * i + 1], c = k[4 * i + 2], d = k[4 * i + 3];
        r.hr1 |= ((b >= a ? 1u : 0u) | (c >= b ? 2u : 0u) | (d >= c ? 4u : 0u) | (a > d ? 8u : 0u)) << (4 * i + shift);
        r.hr2 |= ((c >= a ? 1u : 0u) | (d >= b ? 2u : 0u)) << (4 * i + shift);
        const uint32_t e = k[i], f = k[4 + i], g = k[8 + i], h = k[12 + i];
        r.hc1 |= ((f >= e ? 0x1u : 0u) | (g >= f ? 0x10u : 0u) | (h >= g ? 0x100u : 0u) | (e > h ? 0x1000u : 0u)) << (i + shift);
        r.hc2 |= ((g >= e ? 0x1u : 0u) | (h >= f ? 0x10u : 0u)) << (i + shift);
    }
}

struct alignas(128) TmaEntry {
    CUtensorMap in, out;
    DevProblem p;
    int cchunks;       // items per block row (256 columns each)
};
static_assert(sizeof(TmaEntry) == 384 || sizeof(TmaEntry) == 512, "descriptor records stay 128-byte aligned in tables");

template <int DT, int METHOD, bool HAS_OUT>
__global__ void __launch_bounds__(kWarps * 32, 1)
tma24_kernel(const __grid_constant__ TmaEntry single, const TmaEntry* __restrict__ table, int count, long long total_items,
             double* __restrict__ partials, int* __restrict__ status_out) {
    using G = Geometry<DT>;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned char* wbase = smem_raw + (size_t)warp * G::kWarpBytes;
    unsigned char* stages = wbase;
    unsigned char* mbytes = wbase + G::kStages * G::kStageBytes;          // [4 rows][32 bytes]
    uint64_t* bars = reinterpret_cast<uint64_t*>(mbytes + 128);

    const long long gw = (long long)blockIdx.x * kWarps + warp, nwarps = (long long)gridDim.x * kWarps;
    const long long per = (total_items + nwarps - 1) / nwarps;
    const long long begin = gw * per, end = min(total_items, begin + per);
    const TmaEntry* tab = table ? table : &single;

    if (lane == 0) {
        for (int s = 0; s < G::kStages; ++s) mbar_init(&bars[s], 1);
        fence_mbar_init();
    }
    __syncwarp();

    int status = 0;
    // producer state (lane 0): next item to request and its problem index
    long long next = begin; int next_k = 0;
    auto issue = [&](long long item) {
        while (next_k + 1 < count && tab[next_k + 1].p.item_begin <= item) ++next_k;
        const TmaEntry& e = tab[next_k];
        const long long local = item - e.p.item_begin;
        const int bi = (int)(local / e.cchunks), cj = (int)(local - (long long)bi * e.cchunks);
        const int s = (int)((item - begin) % G::kStages);
        mbar_expect_tx(&bars[s], G::kStageBytes);
        tma_load_2d(stages + s * G::kStageBytes, &e.in, cj * kItemCols, bi * kItemRows, &bars[s]);
    };
    if (lane == 0)
        for (int i = 0; i < G::kStages - 2 && next < end; ++i) issue(next++);

    int k = 0, acc_k = -1;
    float facc = 0.f; double acc = 0.0;
    uint32_t worst = 0;                                                   // largest magnitude pattern seen

    for (long long item = begin; item < end; ++item) {
        const int s = (int)((item - begin) % G::kStages);
        // keep the ring full: the stage being refilled was stored from two items ago
        if (lane == 0 && next < end) {
            if constexpr (HAS_OUT) tma_wait_read<1>();
            issue(next++);
        }
        while (k + 1 < count && tab[k + 1].p.item_begin <= item) ++k;
        const TmaEntry& e = tab[k];
        if (k != acc_k) {
            if (acc_k >= 0) {
                acc += (double)facc; facc = 0.f;
                for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
                if (lane == 0) partials[(long long)acc_k * nwarps + gw] = acc;
            }
            acc = 0.0; acc_k = k;
        }
        const long long local = item - e.p.item_begin;
        const int bi = (int)(local / e.cchunks), cj = (int)(local - (long long)bi * e.cchunks);
        const int col0 = cj * kItemCols + lane * 8;                       // first column of the lane's two blocks
        const uint32_t parity = (uint32_t)(((item - begin) / G::kStages) & 1);
        if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(&bars[s], parity))) {
            // a copy never landed: give the copies still in flight a bounded chance to finish, then stop
            status |= kDevInternal;
            if (lane == 0)
                for (long long j = item + 1; j < next; ++j)
                    mbar_wait_bounded(&bars[(j - begin) % G::kStages], (uint32_t)(((j - begin) / G::kStages) & 1), 1u << 16);
            break;
        }

        unsigned char* stage = stages + s * G::kStageBytes;
        uint32_t raw[4][DT == kF32 ? 8 : 4], ka[16], kb[16];
        load_keys<DT>(stage, lane, raw, ka, kb);
#pragma unroll
        for (int p = 0; p < 16; ++p) worst = max(worst, max(ka[p], kb[p]));

        Rel24 rel = {0, 0, 0, 0, 0, 0};
        relations_scalar(ka, 0, rel);
        relations_scalar(kb, 16, rel);
        complete_relations(rel);
        uint32_t kept = cover_2_4(rel);
        if constexpr (METHOD == kMethodApprox) {
            int rounds = 0;
            while (__any_sync(0xFFFFFFFFu, fill_round_2_4(rel, kept) != 0)) {
                if (++rounds > 4) { status |= kDevInternal; break; }       // a block lacks at most four entries
            }
            const uint32_t sb = short_blocks(kept);
            if (sb & 1) { uint32_t h = kept & 0xFFFFu; if (!swap_fix_2_4(ka, h)) status |= kDevInternal; kept = (kept & 0xFFFF0000u) | h; }
            if (sb & 2) { uint32_t h = kept >> 16; if (!swap_fix_2_4(kb, h)) status |= kDevInternal; kept = (kept & 0xFFFFu) | (h << 16); }
        }
        // blocks past the last column (zero-filled by the copy) contribute nothing
        if (col0 >= e.p.cols) kept = 0;
        else if (col0 + 4 >= e.p.cols) kept &= 0xFFFFu;

        // objective, masked weights, mask bytes
        float s4 = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t na = (kept >> (4 * i)) & 0xFu, nb = (kept >> (16 + 4 * i)) & 0xFu;
            if constexpr (DT == kBF16) {
                uint32_t out[4];
#pragma unroll
                for (int v = 0; v < 4; ++v) {
                    const uint32_t bits = (v < 2 ? na >> (2 * v) : nb >> (2 * (v - 2))) & 3u;
                    const uint32_t m = ((bits & 1u) ? 0x0000FFFFu : 0u) | ((bits & 2u) ? 0xFFFF0000u : 0u);
                    out[v] = raw[i][v] & m;
                    s4 += __uint_as_float((out[v] << 16) & 0x7FFFFFFFu) + __uint_as_float(out[v] & 0x7FFF0000u);
                }
                if constexpr (HAS_OUT)
                    *reinterpret_cast<uint4*>(stage + i * (kItemCols * 2) + lane * 16) = make_uint4(out[0], out[1], out[2], out[3]);
            } else {
                uint32_t out[8];
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    const uint32_t bit = (v < 4 ? na >> v : nb >> (v - 4)) & 1u;
                    out[v] = bit ? raw[i][v] : 0u;
                    s4 += __uint_as_float(out[v] & 0x7FFFFFFFu);
                }
                if constexpr (HAS_OUT) {
                    *reinterpret_cast<uint4*>(stage + i * (kItemCols * 4) + lane * 32) = make_uint4(out[0], out[1], out[2], out[3]);
                    *reinterpret_cast<uint4*>(stage + i * (kItemCols * 4) + lane * 32 + 16) = make_uint4(out[4], out[5], out[6], out[7]);
                }
            }
            mbytes[i * 32 + lane] = (unsigned char)(na | (nb << 4));
        }
        facc += s4;
        if constexpr (HAS_OUT) fence_proxy_async_smem();
        __syncwarp();
        if constexpr (HAS_OUT) {
            if (lane == 0) { tma_store_2d(&e.out, cj * kItemCols, bi * kItemRows, stage); tma_commit(); }
        }
        {   // 4 rows x 8 words of mask
            const int row = lane >> 3, word = cj * 8 + (lane & 7);
            const uint32_t w = *reinterpret_cast<const uint32_t*>(mbytes + row * 32 + (lane & 7) * 4);
            if (word < e.p.wpr) e.p.mask[((long long)bi * kItemRows + row) * e.p.wpr + word] = w;
        }
        __syncwarp();
        if (((item - begin) & 63) == 63) { acc += (double)facc; facc = 0.f; }   // keep the fp32 partial short
    }
    if (lane == 0) tma_wait_all<0>();
    if (acc_k >= 0) {
        acc += (double)facc;
        for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) partials[(long long)acc_k * nwarps + gw] = acc;
    }
    if (worst >= (DT == kF32 ? 0x7F800000u : 0x7F80u)) status |= kDevNonFinite;
    for (int o = 16; o; o >>= 1) status |= __shfl_xor_sync(0xFFFFFFFFu, status, o);
    if (lane == 0 && status && status_out) atomicOr(status_out, status);
}

// objective[k] = sum of the problem's partials in a fixed order (one CTA per problem)
__global__ void __launch_bounds__(256)
reduce_tma_kernel(const __grid_constant__ TmaEntry single, const TmaEntry* __restrict__ table, const double* __restrict__ partials, long long stride) {
    const DevProblem& P = table ? table[blockIdx.x].p : single.p;
    __shared__ double sm[256];
    double s = 0.0;
    for (long long i = threadIdx.x; i < stride; i += 256) s += partials[(long long)blockIdx.x * stride + i];
    sm[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o; o >>= 1) {
        if ((int)threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0 && P.objective) *P.objective = sm[0];
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &p, 12000, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) { cudaGetLastError(); p = nullptr; }
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

bool encode_map(CUtensorMap* m, const void* base, int dtype, long long rows, long long cols, long long ld) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * (dtype == kF32 ? 4 : 2)};
    const cuuint32_t box[2] = {(cuuint32_t)kItemCols, (cuuint32_t)kItemRows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, dtype == kF32 ? CU_TENSOR_MAP_DATA_TYPE_UINT32 : CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(base), dims, strides,
              box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int DT, int METHOD, bool HAS_OUT>
cudaError_t launch_one(const TmaLaunch& a, const TmaEntry& single, const TmaEntry* table) {
    using G = Geometry<DT>;
    const size_t smem = (size_t)kWarps * G::kWarpBytes;
    auto kern = tma24_kernel<DT, METHOD, HAS_OUT>;
    static bool configured = false;        // per instantiation
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    kern<<<a.ctas, kWarps * 32, smem, a.stream>>>(single, table, a.count, a.total_items, a.partials, a.status);
    return cudaGetLastError();
}

}  // namespace

size_t tma_entry_bytes() { return sizeof(TmaEntry); }
int tma_warps_per_cta() { return kWarps; }

bool tma_eligible(const DevProblem& p, int M, int method) {
    if (M != 4 || (method != kMethodApprox && method != kMethodCover)) return false;
    const size_t elem = p.dtype == kF32 ? 4 : 2;
    if ((uintptr_t)p.W % 16 || ((size_t)p.ld * elem) % 16) return false;
    if (p.masked && (uintptr_t)p.masked % 16) return false;
    if (p.rows >= (1ll << 31) || p.cols >= (1ll << 31) || (size_t)p.ld * elem >= (1ull << 40)) return false;
    return encode_fn() != nullptr;
}

// Fills `entries_host` (count TmaEntry records) for problems that all passed tma_eligible().
bool tma_build_entries(const DevProblem* probs, int count, void* entries_host, long long* total_items) {
    TmaEntry* e = static_cast<TmaEntry*>(entries_host);
    long long total = 0;
    for (int k = 0; k < count; ++k) {
        e[k].p = probs[k];
        e[k].cchunks = (int)((probs[k].cols + kItemCols - 1) / kItemCols);
        e[k].p.item_begin = total;
        total += (probs[k].rows / kItemRows) * (long long)e[k].cchunks;
        if (probs[k].rows == 0 || probs[k].cols == 0) { memset(&e[k].in, 0, sizeof(CUtensorMap)); memset(&e[k].out, 0, sizeof(CUtensorMap)); continue; }
        if (!encode_map(&e[k].in, probs[k].W, probs[k].dtype, probs[k].rows, probs[k].cols, probs[k].ld)) return false;
        if (probs[k].masked) {
            if (!encode_map(&e[k].out, probs[k].masked, probs[k].dtype, probs[k].rows, probs[k].cols, probs[k].ld)) return false;
        } else {
            e[k].out = e[k].in;
        }
    }
    *total_items = total;
    return true;
}

// All problems of one launch share dtype and the presence of masked_w_out (the caller groups them).
cudaError_t launch_tma(const TmaLaunch& a) {
    cudaError_t err = cudaMemsetAsync(a.partials, 0, sizeof(double) * (size_t)a.count * (size_t)a.ctas * kWarps, a.stream);
    if (err != cudaSuccess) return err;
    const TmaEntry* host = static_cast<const TmaEntry*>(a.entries_host);
    const TmaEntry* table = static_cast<const TmaEntry*>(a.entries_dev);   // nullptr when count == 1
    if (a.total_items > 0) {
#define TM_DISPATCH(DT, METHOD)                                                                                   \
    err = a.has_out ? launch_one<DT, METHOD, true>(a, host[0], table) : launch_one<DT, METHOD, false>(a, host[0], table)
        if (a.dtype == kF32) { if (a.method == kMethodApprox) TM_DISPATCH(kF32, kMethodApprox); else TM_DISPATCH(kF32, kMethodCover); }
        else { if (a.method == kMethodApprox) TM_DISPATCH(kBF16, kMethodApprox); else TM_DISPATCH(kBF16, kMethodCover); }
#undef TM_DISPATCH
        if (err != cudaSuccess) return err;
    }
    reduce_tma_kernel<<<a.count, 256, 0, a.stream>>>(host[0], table, a.partials, (long long)a.ctas * kWarps);
    return cudaGetLastError();
}

}  // namespace tmask
